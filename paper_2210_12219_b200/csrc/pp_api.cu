// C-ABI of libpp (see include/pp.h) and the host orchestration behind it: validation,
// memory prefix sums, window table, mask lists, launch sequence, result download.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <limits>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "pp_internal.cuh"

using namespace pp;

struct pp_problem {
    int L = 0, k = 0, Lpad = 0, U = 0, elem = 2;
    std::vector<uint64_t> bits, mem, cap, M;
    std::vector<uint32_t> bw, ubw;
    std::vector<int16_t> lo, pair_u;
    unsigned char *d_inputs = nullptr;  // one allocation for all small device arrays
    unsigned char *d_work = nullptr;    // exact-search scratch (own or caller's)
    uint64_t work_bytes = 0;
    bool own_work = false;
    cudaStream_t stream = nullptr;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    pp_solution h_sol_buf{};       // host copy of the result record
    int32_t h_err_buf = 0;
    pp_solution *h_sol = &h_sol_buf;
    pp_solution *d_sol = nullptr;
    int32_t *h_err = &h_err_buf;
    Dev d{};
    bool solved = false, profiled = false;
    int sweep_launches = 0, total_launches = 0, fast_used = 0, pair_levels = 0;
    int force_generic = -1;
    bool profiling = false;             // record events between the phases of a solve
    bool mask_swaps = false;            // the mask list pairs up (see mask_list)
    std::vector<signed char> pair_lvl;  // per level: 1 = two-mask kernel, 0 = one-mask, -1 = not decided yet
};

namespace {

// Mask lists depend on k only: built once per k and process, then copied.  Level j (popcount j)
// lists its masks in revolving-door order: A(n, j) = A(n-1, j), then the masks of A(n-1, j-1) in
// reverse, each with node n-1 added.  Neighbours in that list differ by one node swapped for
// another, which is what the two-mask sweep kernel pairs up.
struct MaskList {
    std::vector<uint32_t> masks, level_off;
    bool swaps = true;  // every two neighbours of a level differ by exactly one swap (checked)
};
void revolving_door(int n, int j, uint32_t add, bool reversed, std::vector<uint32_t> &out)
{
    if (j == 0) { out.push_back(add); return; }
    if (j == n) { out.push_back(add | ((1u << n) - 1u)); return; }
    if (!reversed) {
        revolving_door(n - 1, j, add, false, out);
        revolving_door(n - 1, j - 1, add | (1u << (n - 1)), true, out);
    } else {
        revolving_door(n - 1, j - 1, add | (1u << (n - 1)), false, out);
        revolving_door(n - 1, j, add, true, out);
    }
}
const MaskList &mask_list(int k)
{
    static std::mutex mu;
    static std::map<int, MaskList> cache;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find(k);
    if (it != cache.end()) return it->second;
    MaskList ml;
    const uint32_t nm = 1u << k;
    ml.level_off.assign(k + 2, 0);
    ml.masks.reserve(nm - 1);
    for (int j = 1; j <= k; ++j) {
        ml.level_off[j] = (uint32_t)ml.masks.size();
        revolving_door(k, j, 0u, false, ml.masks);
        for (size_t i = ml.level_off[j] + 1; i < ml.masks.size(); ++i)
            if (__builtin_popcount(ml.masks[i] ^ ml.masks[i - 1]) != 2) ml.swaps = false;
    }
    ml.level_off[k + 1] = (uint32_t)ml.masks.size();
    ml.level_off[0] = 0;
    return cache.emplace(k, std::move(ml)).first->second;
}

// Test hook (pp_debug_fail_alloc): the n-th device allocation from now on reports out of memory
// without asking the driver, so that the out-of-memory paths can be exercised on a healthy device.
std::atomic<int> g_fail_alloc_countdown{0};
bool alloc_should_fail()
{
    int c = g_fail_alloc_countdown.load();
    while (c > 0 && !g_fail_alloc_countdown.compare_exchange_weak(c, c - 1)) {}
    return c == 1;
}

// Device copy of a mask list, uploaded once per (device, k) and kept for the life of the process:
// masks [2^k - 1] followed (256-byte aligned) by level_off [k + 2].
struct DeviceMasks {
    uint32_t *masks = nullptr, *level_off = nullptr;
};
cudaError_t device_masks(int k, const MaskList &ml, DeviceMasks *out)
{
    static std::mutex mu;
    static std::map<std::pair<int, int>, DeviceMasks> cache;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find({dev, k});
    if (it == cache.end()) {
        const size_t mb = (ml.masks.size() * 4 + 255) / 256 * 256, lb = ml.level_off.size() * 4;
        unsigned char *buf = nullptr;
        e = alloc_should_fail() ? cudaErrorMemoryAllocation : cudaMalloc(reinterpret_cast<void **>(&buf), mb + lb);
        if (e != cudaSuccess) return e;
        e = cudaMemcpy(buf, ml.masks.data(), ml.masks.size() * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(buf + mb, ml.level_off.data(), lb, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            cudaFree(buf);
            return e;
        }
        DeviceMasks dm;
        dm.masks = reinterpret_cast<uint32_t *>(buf);
        dm.level_off = reinterpret_cast<uint32_t *>(buf + mb);
        it = cache.emplace(std::make_pair(dev, k), dm).first;
    }
    *out = it->second;
    return cudaSuccess;
}

// Row numbering of the instance-per-lane batch path, per (device, k): rows ordered by (popcount,
// mask, node), the masks listed by (popcount, value).
struct LaneTables {
    uint32_t *rowoff = nullptr, *mlist = nullptr, *moff = nullptr;
};
cudaError_t lane_tables(int k, LaneTables *out)
{
    static std::mutex mu;
    static std::map<std::pair<int, int>, LaneTables> cache;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find({dev, k});
    if (it == cache.end()) {
        const uint32_t nm = 1u << k;
        std::vector<uint32_t> host(2 * (size_t)nm + (size_t)k + 2);
        uint32_t *rowoff = host.data(), *mlist = rowoff + nm, *moff = mlist + nm;
        uint32_t rows = 0, masks = 0;
        for (int pc = 0; pc <= k; ++pc) {
            moff[pc] = masks;
            for (uint32_t S = 0; S < nm; ++S)
                if (__builtin_popcount(S) == pc) {
                    rowoff[S] = rows;
                    rows += (uint32_t)pc;
                    mlist[masks++] = S;
                }
        }
        moff[k + 1] = masks;
        uint32_t *buf = nullptr;
        e = alloc_should_fail() ? cudaErrorMemoryAllocation
                                : cudaMalloc(reinterpret_cast<void **>(&buf), host.size() * 4);
        if (e != cudaSuccess) return e;
        e = cudaMemcpy(buf, host.data(), host.size() * 4, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            cudaFree(buf);
            return e;
        }
        LaneTables lt;
        lt.rowoff = buf;
        lt.mlist = buf + nm;
        lt.moff = buf + 2 * (size_t)nm;
        it = cache.emplace(std::make_pair(dev, k), lt).first;
    }
    *out = it->second;
    return cudaSuccess;
}

// Staging buffers of the host-pointer entry points come from a pool of the library's own that
// keeps its memory between calls (the default pool would hand it back at every synchronisation).
cudaError_t staging_alloc(void **ptr, size_t bytes, cudaStream_t s)
{
    static std::mutex mu;
    static cudaMemPool_t pools[64] = {};
    if (alloc_should_fail()) return cudaErrorMemoryAllocation;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaMalloc(ptr, bytes);
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!pools[dev]) {
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            e = cudaMemPoolCreate(&pools[dev], &props);
            if (e != cudaSuccess) return e;
            unsigned long long keep = ~0ull;
            e = cudaMemPoolSetAttribute(pools[dev], cudaMemPoolAttrReleaseThreshold, &keep);
            if (e != cudaSuccess) return e;
        }
    }
    return cudaMallocFromPoolAsync(ptr, bytes, pools[dev], s);
}

pp_status from_cuda(cudaError_t e)
{
    if (e == cudaSuccess) return PP_OK;
    cudaGetLastError();  // clear the sticky-less error state
    return e == cudaErrorMemoryAllocation ? PP_ERR_NOMEM : PP_ERR_CUDA;
}

#define PP_CUDA(call)                                   \
    do {                                                \
        cudaError_t e__ = (call);                       \
        if (e__ != cudaSuccess) return from_cuda(e__);  \
    } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// instances whose tables share the scratch memory of the instance-per-lane batch path at a time
constexpr int64_t kBatchLanesChunk = 4096;

struct WorkLayout {
    size_t pos, order, gu, cnt, rk, inv, rank, table, total;
};

WorkLayout work_layout(int L, int k, int Lpad, int U, int elem)
{
    WorkLayout w;
    size_t o = 0;
    w.pos = o;   o = align_up(o + (size_t)L * 2, 256);
    w.order = o; o = align_up(o + (size_t)L * 2, 256);
    w.gu = o;    o = align_up(o + (size_t)std::max(U, 1) * L * 8, 256);
    w.cnt = o;   o = align_up(o + (size_t)std::max(U, 1) * L * 4, 256);
    w.rk = o;    o = align_up(o + (size_t)std::max(U, 1) * L * 4, 256);
    w.inv = o;   o = align_up(o + ((size_t)std::max(U, 1) * L + 2) * 4, 256);
    w.rank = o;  o = align_up(o + (size_t)k * k * Lpad * elem, 256);
    w.table = o; o = align_up(o + ((size_t)k << k) * Lpad * elem, 256);
    w.total = o;
    return w;
}

pp_status validate(int32_t L, const uint64_t *bits, const uint64_t *mem, int32_t k,
                   const uint64_t *cap, const uint32_t *bw)
{
    if (!bits || !mem || !cap || !bw) return PP_ERR_ARG;
    if (L < 1 || k < 1) return PP_ERR_ARG;
    if (L > PP_MAX_L || k > PP_MAX_K) return PP_ERR_LIMIT;
    for (int i = 0; i < L; ++i)
        if (bits[i] >= PP_MAX_BITS) return PP_ERR_LIMIT;
    for (int i = 0; i < k * k; ++i)
        if (bw[i] >= PP_MAX_KBPS) return PP_ERR_LIMIT;
    uint64_t acc = 0;
    for (int i = 0; i < L; ++i) {
        if (mem[i] > std::numeric_limits<uint64_t>::max() - acc) return PP_ERR_LIMIT;
        acc += mem[i];
    }
    return PP_OK;
}

void bind_work(pp_problem *p)
{
    WorkLayout w = work_layout(p->L, p->k, p->Lpad, p->U, p->elem);
    unsigned char *b = p->d_work;
    p->d.pos = reinterpret_cast<int16_t *>(b + w.pos);
    p->d.order = reinterpret_cast<int16_t *>(b + w.order);
    p->d.gu = reinterpret_cast<double *>(b + w.gu);
    p->d.cnt = reinterpret_cast<uint32_t *>(b + w.cnt);
    p->d.rk = reinterpret_cast<uint32_t *>(b + w.rk);
    p->d.inv = reinterpret_cast<uint32_t *>(b + w.inv);
    p->d.rank = b + w.rank;
    p->d.table = b + w.table;
    p->d.rank_elems = (uint64_t)p->k * p->k * p->Lpad;
    p->d.table_elems = ((uint64_t)p->k << p->k) * p->Lpad;
}

pp_status ensure_work(pp_problem *p)
{
    if (p->d_work) return PP_OK;
    WorkLayout w = work_layout(p->L, p->k, p->Lpad, p->U, p->elem);
    void *ptr = nullptr;
    if (alloc_should_fail()) return PP_ERR_NOMEM;
    PP_CUDA(cudaMalloc(&ptr, w.total));
    p->d_work = static_cast<unsigned char *>(ptr);
    p->work_bytes = w.total;
    p->own_work = true;
    bind_work(p);
    return PP_OK;
}

pp_status queue_solve(pp_problem *p, pp_solution *sol_dev)
{
    pp_status st = ensure_work(p);
    if (st != PP_OK) return st;
    cudaStream_t s = p->stream;
    bool fast = fast_sweep_supported(p->d);
    if (p->force_generic == 1) fast = false;
    const Dev &d = p->d;
    int launches = 0;
    PP_CUDA(cudaEventRecord(p->ev[0], s));
    PP_CUDA(launch_rank_base(d, s, &launches));
    // an event between two kernels ends the programmatic overlap of their launches: only on request
    if (p->profiling) PP_CUDA(cudaEventRecord(p->ev[1], s));
    int sweep = 0, pairs = 0;
    const int top = std::min(p->k, p->L);
    for (int level = 2; level <= top; ++level) {
        const bool first = level == 2;
        if (fast && p->force_generic != 2) {
            if (p->pair_lvl[level] < 0) p->pair_lvl[level] = pair_sweep_takes(d, level, p->force_generic == 3) ? 1 : 0;
            PP_CUDA(p->pair_lvl[level] ? launch_sweep_pair(d, level, s, first) : launch_sweep_fast(d, level, s, first));
            pairs += p->pair_lvl[level];
        } else {
            PP_CUDA(fast ? launch_sweep_fast(d, level, s, first) : launch_sweep_generic(d, level, s));
        }
        ++sweep;
    }
    if (p->profiling) PP_CUDA(cudaEventRecord(p->ev[2], s));
    PP_CUDA(launch_finalize(d, sol_dev, s, true));
    PP_CUDA(cudaEventRecord(p->ev[3], s));
    p->sweep_launches = sweep;
    p->pair_levels = pairs;
    p->total_launches = launches + sweep + 1;
    p->fast_used = fast ? (p->d.fast_meta ? 1 : 2) : 0;
    p->solved = true;
    p->profiled = p->profiling;
    return PP_OK;
}

}  // namespace

extern "C" {

const char *pp_status_str(pp_status s)
{
    switch (s) {
        case PP_OK: return "ok";
        case PP_INFEASIBLE: return "infeasible: no plan exists";
        case PP_ERR_ARG: return "bad argument";
        case PP_ERR_LIMIT: return "size or value above the library limits";
        case PP_ERR_NOMEM: return "out of memory";
        case PP_ERR_CUDA: return "CUDA runtime error";
        case PP_ERR_TIMEOUT: return "timeout";
    }
    return "unknown status";
}

pp_status pp_problem_create(int32_t L, const uint64_t *layer_out_bits,
                            const uint64_t *layer_mem_bytes, int32_t k,
                            const uint64_t *node_mem_bytes, const uint32_t *bw_kbps,
                            pp_problem **out)
{
    if (!out) return PP_ERR_ARG;
    pp_status st = validate(L, layer_out_bits, layer_mem_bytes, k, node_mem_bytes, bw_kbps);
    if (st != PP_OK) return st;
    pp_problem *p = new (std::nothrow) pp_problem();
    if (!p) return PP_ERR_NOMEM;
    try {
        p->L = L;
        p->k = k;
        p->bits.assign(layer_out_bits, layer_out_bits + L);
        p->mem.assign(layer_mem_bytes, layer_mem_bytes + L);
        p->cap.assign(node_mem_bytes, node_mem_bytes + k);
        p->bw.assign(bw_kbps, bw_kbps + (size_t)k * k);
        // memory prefix sums: segment first..last needs M[last+1] - M[first] bytes
        p->M.assign(L + 1, 0);
        for (int i = 0; i < L; ++i) p->M[i + 1] = p->M[i] + p->mem[i];
        // window table: lo[w][c'] = earliest previous cut c >= 0 such that layers c+1..c' fit on
        // w; c' itself when not even layer c' alone fits.  Non-decreasing in c'.
        p->lo.assign((size_t)k * L, 0);
        for (int w = 0; w < k; ++w) {
            int c = 0;
            for (int c2 = 0; c2 < L; ++c2) {
                while (c < c2 && p->M[c2 + 1] - p->M[c + 1] > p->cap[w]) ++c;
                p->lo[(size_t)w * L + c2] = (int16_t)c;
            }
        }
        // distinct usable bandwidths
        std::map<uint32_t, int> seen;
        p->pair_u.assign((size_t)k * k, -1);
        for (int v = 0; v < k; ++v)
            for (int w = 0; w < k; ++w) {
                uint32_t b = p->bw[(size_t)v * k + w];
                if (v == w || b == 0) continue;
                auto it = seen.find(b);
                if (it == seen.end()) {
                    it = seen.emplace(b, (int)p->ubw.size()).first;
                    p->ubw.push_back(b);
                }
                p->pair_u[(size_t)v * k + w] = (int16_t)it->second;
            }
        p->U = (int)p->ubw.size();
        if (p->ubw.empty()) p->ubw.push_back(0);  // keep the upload non-empty; U stays 0
        // 16-bit ranks when 0, 1..L*U and the +inf code all fit
        p->elem = ((uint64_t)L * (uint64_t)std::max(p->U, 1) + 1 <= 65534) ? 2 : 4;
        const int per32 = 32 / p->elem;
        p->Lpad = (L + per32 - 1) / per32 * per32;
        // masks by (popcount, value)
        const MaskList &ml = mask_list(k);
        p->mask_swaps = ml.swaps;
        p->pair_lvl.assign(k + 2, -1);
    } catch (const std::bad_alloc &) {
        delete p;
        return PP_ERR_NOMEM;
    }

    // constants of the register-tiled sweep, when the instance is inside its envelope
    std::vector<unsigned char> fmeta;
    bool has_fast = false;
    try {
        fmeta.resize(fast_meta_bytes());
        has_fast = p->elem == 2 && p->Lpad <= 240 && k >= 2 &&
                   fast_meta_build(L, k, p->lo.data(), fmeta.data());
    } catch (const std::bad_alloc &) {
        delete p;
        return PP_ERR_NOMEM;
    }
    std::vector<unsigned char> pmeta;
    try {
        if (has_fast && p->mask_swaps) {
            pmeta.resize(pair_meta_bytes());
            if (!pair_meta_build(L, k, p->lo.data(), pmeta.data())) pmeta.clear();
        }
    } catch (const std::bad_alloc &) {
        delete p;
        return PP_ERR_NOMEM;
    }
    std::vector<uint32_t> gmeta;
    try {
        if (!has_fast && p->elem == 2 && p->Lpad <= 240 && k >= 2) {
            gmeta.resize((size_t)k * p->Lpad);
            p->d.gen_levels = gen_meta_build(L, k, p->Lpad, p->lo.data(), gmeta.data());
        }
    } catch (const std::bad_alloc &) {
        delete p;
        return PP_ERR_NOMEM;
    }
    // upload the small arrays in one allocation
    struct Part { const void *src; size_t bytes; size_t off; };
    std::vector<Part> parts = {
        {p->bits.data(), p->bits.size() * 8, 0},       {p->M.data(), p->M.size() * 8, 0},
        {p->cap.data(), p->cap.size() * 8, 0},         {p->bw.data(), p->bw.size() * 4, 0},
        {p->lo.data(), p->lo.size() * 2, 0},           {p->pair_u.data(), p->pair_u.size() * 2, 0},
        {p->ubw.data(), p->ubw.size() * 4, 0},
        {nullptr, 0, 0} /* masks: shared */,           {nullptr, 0, 0} /* level_off: shared */,
        {nullptr, 8, 0} /* best */,                    {nullptr, 4, 0} /* err */,
        {nullptr, sizeof(pp_solution), 0} /* solution */,
        {fmeta.data(), fmeta.size(), 0},
        {gmeta.data(), gmeta.size() * 4, 0},
        {pmeta.data(), pmeta.size(), 0}};
    size_t total = 0;
    for (auto &q : parts) { q.off = total; total = align_up(total + q.bytes, 256); }
    // one staging buffer, one copy: the parts are small and a copy per part costs more than the bytes
    std::vector<unsigned char> staging;
    try {
        staging.assign(total, 0);
    } catch (const std::bad_alloc &) {
        delete p;
        return PP_ERR_NOMEM;
    }
    for (auto &q : parts)
        if (q.src && q.bytes) std::memcpy(staging.data() + q.off, q.src, q.bytes);
    DeviceMasks dmasks;
    cudaError_t e = device_masks(k, mask_list(k), &dmasks);
    if (e == cudaSuccess) e = staging_alloc(reinterpret_cast<void **>(&p->d_inputs), total, nullptr);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_inputs, staging.data(), total, cudaMemcpyHostToDevice);
    for (int i = 0; i < 4 && e == cudaSuccess; ++i) e = cudaEventCreate(&p->ev[i]);
    if (e != cudaSuccess) {
        pp_status rc = from_cuda(e);
        pp_problem_destroy(p);
        return rc;
    }
    unsigned char *b = p->d_inputs;
    Dev &d = p->d;
    d.L = L; d.k = k; d.Lpad = p->Lpad; d.U = p->U; d.elem = p->elem;
    d.bits = reinterpret_cast<uint64_t *>(b + parts[0].off);
    d.M = reinterpret_cast<uint64_t *>(b + parts[1].off);
    d.cap = reinterpret_cast<uint64_t *>(b + parts[2].off);
    d.bw = reinterpret_cast<uint32_t *>(b + parts[3].off);
    d.lo = reinterpret_cast<int16_t *>(b + parts[4].off);
    d.pair_u = reinterpret_cast<int16_t *>(b + parts[5].off);
    d.ubw = reinterpret_cast<uint32_t *>(b + parts[6].off);
    d.masks = dmasks.masks;  // shared by every problem of this k on this device
    d.level_off = dmasks.level_off;
    d.best = reinterpret_cast<unsigned long long *>(b + parts[9].off);
    d.err = reinterpret_cast<int32_t *>(b + parts[10].off);
    p->d_sol = reinterpret_cast<pp_solution *>(b + parts[11].off);
    d.fast_meta = has_fast ? b + parts[12].off : nullptr;
    d.gen_meta = gmeta.empty() ? nullptr : reinterpret_cast<uint32_t *>(b + parts[13].off);
    d.pair_meta = pmeta.empty() ? nullptr : b + parts[14].off;
    *out = p;
    return PP_OK;
}

void pp_problem_destroy(pp_problem *p)
{
    if (!p) return;
    if (p->own_work && p->d_work) cudaFree(p->d_work);
    if (p->d_inputs) cudaFreeAsync(p->d_inputs, p->stream);  // ordered after the problem's queued work
    for (auto &e : p->ev)
        if (e) cudaEventDestroy(e);
    delete p;
}

pp_status pp_problem_set_stream(pp_problem *p, void *cuda_stream)
{
    if (!p) return PP_ERR_ARG;
    p->stream = static_cast<cudaStream_t>(cuda_stream);
    return PP_OK;
}

pp_status pp_problem_workspace_bytes(const pp_problem *p, uint64_t *bytes)
{
    if (!p || !bytes) return PP_ERR_ARG;
    *bytes = work_layout(p->L, p->k, p->Lpad, p->U, p->elem).total;
    return PP_OK;
}

pp_status pp_problem_set_workspace(pp_problem *p, void *device_buffer, uint64_t bytes)
{
    if (!p || !device_buffer) return PP_ERR_ARG;
    if (reinterpret_cast<uintptr_t>(device_buffer) % 256) return PP_ERR_ARG;
    if (bytes < work_layout(p->L, p->k, p->Lpad, p->U, p->elem).total) return PP_ERR_NOMEM;
    if (p->own_work && p->d_work) {
        cudaStreamSynchronize(p->stream);
        cudaFree(p->d_work);
    }
    p->d_work = static_cast<unsigned char *>(device_buffer);
    p->work_bytes = bytes;
    p->own_work = false;
    p->solved = false;
    bind_work(p);
    return PP_OK;
}

pp_status pp_problem_force_generic(pp_problem *p, int32_t mode)
{
    if (!p || mode < -1 || mode > 3) return PP_ERR_ARG;
    p->force_generic = mode;
    p->pair_lvl.assign(p->k + 2, -1);
    return PP_OK;
}

pp_status pp_problem_set_profiling(pp_problem *p, int32_t on)
{
    if (!p) return PP_ERR_ARG;
    p->profiling = on != 0;
    return PP_OK;
}

pp_status pp_solve_exact_dev(pp_problem *p, pp_solution *solution_dev)
{
    if (!p || !solution_dev) return PP_ERR_ARG;
    return queue_solve(p, solution_dev);
}

pp_status pp_solve_exact(pp_problem *p, double *beta_ms, int32_t *m, int32_t *cuts,
                         int32_t *placement)
{
    if (!p || !beta_ms || !m || !placement || (!cuts && p->k > 1)) return PP_ERR_ARG;
    PP_CUDA(cudaMemsetAsync(p->d.err, 0, sizeof(int32_t), p->stream));
    pp_status st = queue_solve(p, p->d_sol);
    if (st != PP_OK) return st;
    PP_CUDA(cudaMemcpyAsync(p->h_sol, p->d_sol, sizeof(pp_solution), cudaMemcpyDeviceToHost, p->stream));
    PP_CUDA(cudaMemcpyAsync(p->h_err, p->d.err, sizeof(int32_t), cudaMemcpyDeviceToHost, p->stream));
    PP_CUDA(cudaStreamSynchronize(p->stream));
    if (*p->h_err) return PP_ERR_CUDA;
    *beta_ms = p->h_sol->beta_ms;
    *m = p->h_sol->m;
    for (int j = 0; j < p->k - 1; ++j) cuts[j] = p->h_sol->cuts[j];
    for (int j = 0; j < p->k; ++j) placement[j] = p->h_sol->placement[j];
    return static_cast<pp_status>(p->h_sol->status);
}

pp_status pp_last_solve_profile(pp_problem *p, pp_profile *out)
{
    if (!p || !out || !p->solved) return PP_ERR_ARG;
    PP_CUDA(cudaStreamSynchronize(p->stream));
    out->ms_rank = out->ms_sweep = out->ms_finalize = 0.0f;
    if (p->profiled) {
        PP_CUDA(cudaEventElapsedTime(&out->ms_rank, p->ev[0], p->ev[1]));
        PP_CUDA(cudaEventElapsedTime(&out->ms_sweep, p->ev[1], p->ev[2]));
        PP_CUDA(cudaEventElapsedTime(&out->ms_finalize, p->ev[2], p->ev[3]));
    }
    PP_CUDA(cudaEventElapsedTime(&out->ms_total, p->ev[0], p->ev[3]));
    out->sweep_launches = p->sweep_launches;
    out->total_launches = p->total_launches;
    out->state_bytes = p->elem;
    out->fast_path = p->fast_used;
    out->pair_levels = p->pair_levels;
    return PP_OK;
}

pp_status pp_eval_plans_dev(pp_problem *p, int64_t B, const uint8_t *nseg, const int32_t *ends,
                            const int32_t *nodes, double *beta_ms, uint8_t *plan_status)
{
    if (!p || B < 0) return PP_ERR_ARG;
    if (B == 0) return PP_OK;
    if (!nseg || !ends || !nodes || !beta_ms || !plan_status) return PP_ERR_ARG;
    PP_CUDA(launch_eval(p->d, B, nseg, ends, nodes, beta_ms, plan_status, p->stream));
    return PP_OK;
}

pp_status pp_eval_plans(pp_problem *p, int64_t B, const uint8_t *nseg, const int32_t *ends,
                        const int32_t *nodes, double *beta_ms, uint8_t *plan_status)
{
    if (!p || B < 0) return PP_ERR_ARG;
    if (B == 0) return PP_OK;
    if (!nseg || !ends || !nodes || !beta_ms || !plan_status) return PP_ERR_ARG;
    const size_t k = p->k;
    const size_t b_nseg = (size_t)B, b_rows = (size_t)B * k * 4, b_beta = (size_t)B * 8;
    size_t o_ends = align_up(b_nseg, 256), o_nodes = align_up(o_ends + b_rows, 256);
    size_t o_beta = align_up(o_nodes + b_rows, 256), o_st = align_up(o_beta + b_beta, 256);
    size_t total = o_st + (size_t)B;
    unsigned char *buf = nullptr;
    cudaStream_t s = p->stream;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), total, s));
    cudaError_t e = cudaMemcpyAsync(buf, nseg, b_nseg, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(buf + o_ends, ends, b_rows, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(buf + o_nodes, nodes, b_rows, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = launch_eval(p->d, B, buf, reinterpret_cast<int32_t *>(buf + o_ends),
                        reinterpret_cast<int32_t *>(buf + o_nodes),
                        reinterpret_cast<double *>(buf + o_beta), buf + o_st, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(beta_ms, buf + o_beta, b_beta, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(plan_status, buf + o_st, (size_t)B, cudaMemcpyDeviceToHost, s);
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

pp_status pp_eval_plans_packed_dev(pp_problem *p, int64_t B, int64_t total, const uint8_t *nseg,
                                   const uint32_t *plan_off, const uint16_t *ends, const uint8_t *nodes,
                                   double *beta_ms, uint8_t *plan_status)
{
    if (!p || B < 0 || total < 0) return PP_ERR_ARG;
    if (B == 0) return PP_OK;
    if (!nseg || !plan_off || !beta_ms || !plan_status || ((!ends || !nodes) && total > 0)) return PP_ERR_ARG;
    PP_CUDA(launch_eval_packed(p->d, B, total, nseg, plan_off, ends, nodes, beta_ms, plan_status, p->stream));
    return PP_OK;
}

pp_status pp_eval_plans_packed(pp_problem *p, int64_t B, int64_t total, const uint8_t *nseg,
                               const uint32_t *plan_off, const uint16_t *ends, const uint8_t *nodes,
                               double *beta_ms, uint8_t *plan_status)
{
    if (!p || B < 0 || total < 0) return PP_ERR_ARG;
    if (B == 0) return PP_OK;
    if (!nseg || !plan_off || !beta_ms || !plan_status || ((!ends || !nodes) && total > 0)) return PP_ERR_ARG;
    const size_t nB = (size_t)B, nT = (size_t)total;
    const size_t o_off = align_up(nB, 256), o_ends = align_up(o_off + (nB + 1) * 4, 256);
    const size_t o_nodes = align_up(o_ends + nT * 2, 256), o_beta = align_up(o_nodes + nT, 256);
    const size_t o_st = align_up(o_beta + nB * 8, 256), bytes = o_st + nB;
    unsigned char *buf = nullptr;
    cudaStream_t s = p->stream;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), bytes, s));
    cudaError_t e = cudaMemcpyAsync(buf, nseg, nB, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(buf + o_off, plan_off, (nB + 1) * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && nT) e = cudaMemcpyAsync(buf + o_ends, ends, nT * 2, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && nT) e = cudaMemcpyAsync(buf + o_nodes, nodes, nT, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = launch_eval_packed(p->d, B, total, buf, reinterpret_cast<uint32_t *>(buf + o_off),
                               reinterpret_cast<uint16_t *>(buf + o_ends), buf + o_nodes,
                               reinterpret_cast<double *>(buf + o_beta), buf + o_st, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(beta_ms, buf + o_beta, nB * 8, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(plan_status, buf + o_st, nB, cudaMemcpyDeviceToHost, s);
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

pp_status pp_random_plans_dev(pp_problem *p, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                              int32_t *nodes)
{
    if (!p || P < 0) return PP_ERR_ARG;
    if (P == 0) return PP_OK;
    if (!draws || !nseg || !ends || !nodes) return PP_ERR_ARG;
    PP_CUDA(launch_random_plans(p->d, P, draws, nseg, ends, nodes, p->stream));
    return PP_OK;
}

pp_status pp_random_plans(pp_problem *p, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                          int32_t *nodes)
{
    if (!p || P < 0) return PP_ERR_ARG;
    if (P == 0) return PP_OK;
    if (!draws || !nseg || !ends || !nodes) return PP_ERR_ARG;
    const size_t k = p->k;
    const size_t b_draws = (size_t)P * 2 * k * 4, b_rows = (size_t)P * k * 4;
    const size_t o_ends = align_up(b_draws, 256), o_nodes = align_up(o_ends + b_rows, 256);
    const size_t o_nseg = align_up(o_nodes + b_rows, 256), total = o_nseg + (size_t)P;
    unsigned char *buf = nullptr;
    cudaStream_t s = p->stream;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), total, s));
    cudaError_t e = cudaMemcpyAsync(buf, draws, b_draws, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = launch_random_plans(p->d, P, reinterpret_cast<uint32_t *>(buf), buf + o_nseg,
                                reinterpret_cast<int32_t *>(buf + o_ends),
                                reinterpret_cast<int32_t *>(buf + o_nodes), s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(nseg, buf + o_nseg, (size_t)P, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ends, buf + o_ends, b_rows, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(nodes, buf + o_nodes, b_rows, cudaMemcpyDeviceToHost, s);
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

pp_status pp_solve_exact_batch_dev(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                                   const uint64_t *mem, const uint64_t *node_mem,
                                   const uint32_t *bw, double *beta_ms, int32_t *m, int32_t *cuts,
                                   int32_t *placement, int8_t *status, void *cuda_stream)
{
    if (B < 0 || L < 1 || k < 1) return PP_ERR_ARG;
    if (L > PP_MAX_L || k > PP_MAX_K) return PP_ERR_LIMIT;
    if (B == 0) return PP_OK;
    if (!out_bits || !mem || !node_mem || !bw || !beta_ms || !m || !placement || !status ||
        (!cuts && k > 1))
        return PP_ERR_ARG;
    int dev = 0, max_sm = 0;
    PP_CUDA(cudaGetDevice(&dev));
    PP_CUDA(cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    if (batch_smem_bytes(L, k) + 1024 > (size_t)max_sm) return PP_ERR_LIMIT;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (!batch_lanes_takes(B, L, k)) {
        PP_CUDA(launch_batch(B, L, k, out_bits, mem, node_mem, bw, beta_ms, m, cuts, placement, status, s));
        return PP_OK;
    }
    // Instance-per-lane path: the tables of a chunk of instances live in scratch memory from the
    // library's pool, ordered on the caller's stream; chunks follow one another on that stream.
    LaneTables lt;
    PP_CUDA(lane_tables(k, &lt));
    const int64_t chunk = std::min<int64_t>(B, kBatchLanesChunk);
    const size_t G = (size_t)((chunk + 31) / 32);
    BatchLanes t;
    t.LH = batch_lanes_words(L);
    t.rows = (uint32_t)k << (k - 1);
    t.rowoff = lt.rowoff;
    t.mlist = lt.mlist;
    t.moff = lt.moff;
    const size_t line = (size_t)t.LH * 32 * sizeof(uint32_t);
    const size_t b_table = G * t.rows * line, b_rank = G * (size_t)(k * k) * line, b_len = G * (size_t)k * line;
    const size_t b_win = 2 * b_len;
    const size_t b_key = G * 32 * sizeof(unsigned long long), b_flag = align_up(G * 32, 256), b_err = 256;
    unsigned char *buf = nullptr;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), b_table + b_rank + b_len + b_win + b_key + b_flag + b_err, s));
    t.table = reinterpret_cast<uint32_t *>(buf);
    t.rank = reinterpret_cast<uint32_t *>(buf + b_table);
    t.len = reinterpret_cast<uint32_t *>(buf + b_table + b_rank);
    t.win = reinterpret_cast<uint32_t *>(buf + b_table + b_rank + b_len);
    t.key = reinterpret_cast<unsigned long long *>(buf + b_table + b_rank + b_len + b_win);
    t.flag = reinterpret_cast<int8_t *>(buf + b_table + b_rank + b_len + b_win + b_key);
    t.err = reinterpret_cast<int32_t *>(buf + b_table + b_rank + b_len + b_win + b_key + b_flag);
    t.table_words = b_table / 4;
    t.rank_words = b_rank / 4;
    t.len_words = b_len / 4;
    t.win_words = b_win / 4;
#ifdef PP_DEBUG_BOUNDS
    {  // the bounds-checking build records violations here; k_lanes_back turns them into PP_ERR_CUDA
        cudaError_t ez = cudaMemsetAsync(t.err, 0, sizeof(int32_t), s);
        if (ez != cudaSuccess) {
            cudaFreeAsync(buf, s);
            return from_cuda(ez);
        }
    }
#endif
    cudaError_t e = cudaSuccess;
    for (int64_t b0 = 0; b0 < B && e == cudaSuccess; b0 += chunk) {
        const int64_t n = std::min<int64_t>(chunk, B - b0);
        e = launch_batch_prep(n, L, k, out_bits + b0 * L, mem + b0 * L, node_mem + b0 * k, bw + b0 * k * k, t, s);
        if (e == cudaSuccess)
            e = launch_batch_lanes(n, L, k, out_bits + b0 * L, bw + b0 * k * k, t, beta_ms + b0, m + b0,
                                   cuts ? cuts + b0 * (k - 1) : nullptr, placement + b0 * k, status + b0, s);
    }
    cudaFreeAsync(buf, s);
    PP_CUDA(e);
    return PP_OK;
}

// Host-pointer form of a batched entry point: stage the inputs, run the device-pointer form on
// the legacy default stream, bring the results back.
typedef pp_status (*batch_dev_fn)(int64_t, int32_t, int32_t, const uint64_t *, const uint64_t *,
                                  const uint64_t *, const uint32_t *, double *, int32_t *, int32_t *,
                                  int32_t *, int8_t *, void *);

static pp_status batch_from_host(batch_dev_fn run_dev, int64_t B, int32_t L, int32_t k,
                                 const uint64_t *out_bits, const uint64_t *mem, const uint64_t *node_mem,
                                 const uint32_t *bw, double *beta_ms, int32_t *m, int32_t *cuts,
                                 int32_t *placement, int8_t *status)
{
    if (B < 0 || L < 1 || k < 1) return PP_ERR_ARG;
    if (L > PP_MAX_L || k > PP_MAX_K) return PP_ERR_LIMIT;
    if (B == 0) return PP_OK;
    if (!out_bits || !mem || !node_mem || !bw || !beta_ms || !m || !placement || !status ||
        (!cuts && k > 1))
        return PP_ERR_ARG;
    const size_t nB = (size_t)B;
    const size_t sz[9] = {nB * L * 8, nB * L * 8, nB * k * 8, nB * k * k * 4, nB * 8,
                          nB * 4,     nB * (size_t)std::max(k - 1, 1) * 4, nB * k * 4, nB};
    size_t off[10];
    off[0] = 0;
    for (int i = 0; i < 9; ++i) off[i + 1] = align_up(off[i] + sz[i], 256);
    unsigned char *buf = nullptr;
    cudaStream_t s = nullptr;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), off[9], s));
    const void *src[4] = {out_bits, mem, node_mem, bw};
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < 4 && e == cudaSuccess; ++i)
        e = cudaMemcpyAsync(buf + off[i], src[i], sz[i], cudaMemcpyHostToDevice, s);
    pp_status st = PP_OK;
    if (e == cudaSuccess)
        st = run_dev(B, L, k, reinterpret_cast<uint64_t *>(buf + off[0]),
                     reinterpret_cast<uint64_t *>(buf + off[1]), reinterpret_cast<uint64_t *>(buf + off[2]),
                     reinterpret_cast<uint32_t *>(buf + off[3]), reinterpret_cast<double *>(buf + off[4]),
                     reinterpret_cast<int32_t *>(buf + off[5]), reinterpret_cast<int32_t *>(buf + off[6]),
                     reinterpret_cast<int32_t *>(buf + off[7]), reinterpret_cast<int8_t *>(buf + off[8]), s);
    if (e == cudaSuccess && st == PP_OK) {
        void *dst[5] = {beta_ms, m, cuts, placement, status};
        for (int i = 0; i < 5 && e == cudaSuccess; ++i) {
            if (!dst[i]) continue;
            size_t n = (i == 2) ? nB * (size_t)(k - 1) * 4 : sz[4 + i];
            if (n) e = cudaMemcpyAsync(dst[i], buf + off[4 + i], n, cudaMemcpyDeviceToHost, s);
        }
    }
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (st != PP_OK) return st;
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

pp_status pp_solve_exact_batch(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                               const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                               double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement,
                               int8_t *status)
{
    return batch_from_host(pp_solve_exact_batch_dev, B, L, k, out_bits, mem, node_mem, bw, beta_ms, m, cuts,
                           placement, status);
}

pp_status pp_greedy_batch_dev(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                              const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                              double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement,
                              int8_t *status, void *cuda_stream)
{
    if (B < 0 || L < 1 || k < 1) return PP_ERR_ARG;
    if (L > PP_MAX_L || k > PP_MAX_K) return PP_ERR_LIMIT;
    if (B == 0) return PP_OK;
    if (!out_bits || !mem || !node_mem || !bw || !beta_ms || !m || !placement || !status ||
        (!cuts && k > 1))
        return PP_ERR_ARG;
    PP_CUDA(launch_greedy(B, L, k, out_bits, mem, node_mem, bw, beta_ms, m, cuts, placement, status,
                          static_cast<cudaStream_t>(cuda_stream)));
    return PP_OK;
}

pp_status pp_greedy_batch(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                          const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                          double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement, int8_t *status)
{
    return batch_from_host(pp_greedy_batch_dev, B, L, k, out_bits, mem, node_mem, bw, beta_ms, m, cuts,
                           placement, status);
}

pp_status pp_partition_minsum_batch_dev(int64_t B, int32_t L, const uint64_t *cut_weight, const uint64_t *mem,
                                        const uint64_t *kappa, int32_t cap_seg, uint64_t *cost, int32_t *m,
                                        int32_t *cuts, uint64_t *sizes, int8_t *status, void *cuda_stream)
{
    if (B < 0 || L < 1 || cap_seg < 0) return PP_ERR_ARG;
    if (L > PP_MAX_L) return PP_ERR_LIMIT;
    if (B == 0) return PP_OK;
    if (!cut_weight || !mem || !kappa || !cost || !m || !status || (!cuts && cap_seg > 0)) return PP_ERR_ARG;
    PP_CUDA(launch_partition_minsum(B, L, cap_seg, cut_weight, mem, kappa, cost, m, cuts, sizes, status,
                                    static_cast<cudaStream_t>(cuda_stream)));
    return PP_OK;
}

pp_status pp_partition_minsum_batch(int64_t B, int32_t L, const uint64_t *cut_weight, const uint64_t *mem,
                                    const uint64_t *kappa, int32_t cap_seg, uint64_t *cost, int32_t *m,
                                    int32_t *cuts, uint64_t *sizes, int8_t *status)
{
    if (B < 0 || L < 1 || cap_seg < 0) return PP_ERR_ARG;
    if (L > PP_MAX_L) return PP_ERR_LIMIT;
    if (B == 0) return PP_OK;
    if (!cut_weight || !mem || !kappa || !cost || !m || !status || (!cuts && cap_seg > 0)) return PP_ERR_ARG;
    const size_t nB = (size_t)B, rows = nB * (size_t)std::max(cap_seg, 1);
    const size_t sz[8] = {nB * L * 8, nB * L * 8, nB * 8, nB * 8, nB * 4, rows * 4, rows * 8, nB};
    size_t off[9];
    off[0] = 0;
    for (int i = 0; i < 8; ++i) off[i + 1] = align_up(off[i] + sz[i], 256);
    unsigned char *buf = nullptr;
    cudaStream_t s = nullptr;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), off[8], s));
    const void *src[3] = {cut_weight, mem, kappa};
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < 3 && e == cudaSuccess; ++i)
        e = cudaMemcpyAsync(buf + off[i], src[i], sz[i], cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = launch_partition_minsum(B, L, cap_seg, reinterpret_cast<uint64_t *>(buf + off[0]),
                                    reinterpret_cast<uint64_t *>(buf + off[1]), reinterpret_cast<uint64_t *>(buf + off[2]),
                                    reinterpret_cast<uint64_t *>(buf + off[3]), reinterpret_cast<int32_t *>(buf + off[4]),
                                    reinterpret_cast<int32_t *>(buf + off[5]), reinterpret_cast<uint64_t *>(buf + off[6]),
                                    reinterpret_cast<int8_t *>(buf + off[7]), s);
    if (e == cudaSuccess) {
        void *dst[5] = {cost, m, cuts, sizes, status};
        const size_t n[5] = {sz[3], sz[4], nB * (size_t)cap_seg * 4, nB * (size_t)cap_seg * 8, sz[7]};
        for (int i = 0; i < 5 && e == cudaSuccess; ++i)
            if (dst[i] && n[i]) e = cudaMemcpyAsync(dst[i], buf + off[3 + i], n[i], cudaMemcpyDeviceToHost, s);
    }
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

pp_status pp_kpath_colour_batch_dev(int32_t n, const uint32_t *bw_kbps, int64_t Q, int32_t kk,
                                    const uint32_t *threshold, const int32_t *start, const int32_t *end,
                                    const uint64_t *alive, const uint8_t *colours, uint8_t *found, int32_t *path,
                                    void *cuda_stream)
{
    if (n < 1 || kk < 1 || Q < 0) return PP_ERR_ARG;
    if (n > PP_KPATH_MAX_N || kk > PP_KPATH_MAX_K) return PP_ERR_LIMIT;
    if (Q == 0) return PP_OK;
    if (!bw_kbps || !threshold || !start || !end || !alive || !colours || !found || !path) return PP_ERR_ARG;
    PP_CUDA(launch_kpath(n, kk, Q, bw_kbps, threshold, start, end, reinterpret_cast<const unsigned long long *>(alive),
                         colours, found, path, static_cast<cudaStream_t>(cuda_stream)));
    return PP_OK;
}

pp_status pp_kpath_colour_batch(int32_t n, const uint32_t *bw_kbps, int64_t Q, int32_t kk, const uint32_t *threshold,
                                const int32_t *start, const int32_t *end, const uint64_t *alive,
                                const uint8_t *colours, uint8_t *found, int32_t *path)
{
    if (n < 1 || kk < 1 || Q < 0) return PP_ERR_ARG;
    if (n > PP_KPATH_MAX_N || kk > PP_KPATH_MAX_K) return PP_ERR_LIMIT;
    if (Q == 0) return PP_OK;
    if (!bw_kbps || !threshold || !start || !end || !alive || !colours || !found || !path) return PP_ERR_ARG;
    const size_t nQ = (size_t)Q;
    const size_t sz[9] = {(size_t)n * n * 4, nQ * 4, nQ * 4, nQ * 4, nQ * 8, nQ * n, nQ, nQ * kk * 4, 0};
    size_t off[9];
    off[0] = 0;
    for (int i = 0; i < 8; ++i) off[i + 1] = align_up(off[i] + sz[i], 256);
    unsigned char *buf = nullptr;
    cudaStream_t s = nullptr;
    PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), off[8], s));
    const void *src[6] = {bw_kbps, threshold, start, end, alive, colours};
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < 6 && e == cudaSuccess; ++i)
        e = cudaMemcpyAsync(buf + off[i], src[i], sz[i], cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)
        e = launch_kpath(n, kk, Q, reinterpret_cast<uint32_t *>(buf + off[0]), reinterpret_cast<uint32_t *>(buf + off[1]),
                         reinterpret_cast<int32_t *>(buf + off[2]), reinterpret_cast<int32_t *>(buf + off[3]),
                         reinterpret_cast<unsigned long long *>(buf + off[4]), buf + off[5], buf + off[6],
                         reinterpret_cast<int32_t *>(buf + off[7]), s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(found, buf + off[6], sz[6], cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(path, buf + off[7], sz[7], cudaMemcpyDeviceToHost, s);
    cudaFreeAsync(buf, s);
    cudaError_t e2 = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return from_cuda(e);
    return from_cuda(e2);
}

// Placement stage of the paper's heuristic (Section 3.2.2, Algorithms 2 and 3), orchestrated on the
// host: classes of the cut sizes, runs of cuts per class, and for every run a bisection over the
// sorted link bandwidths whose probes are batches of colour-coding k-path queries on the device (one
// query per trial colouring).
pp_status pp_kpath_matching(int32_t n, const uint32_t *bw_kbps, int32_t n_cuts, const uint64_t *sizes,
                            int32_t n_classes, int32_t trials, const uint32_t *draws, int32_t *nodes,
                            uint32_t *cut_threshold, void *cuda_stream)
{
    if (n < 1 || n_cuts < 0 || n_classes < 1 || trials < 1) return PP_ERR_ARG;
    if (!bw_kbps || !draws || !nodes || (!sizes && n_cuts > 0)) return PP_ERR_ARG;
    if (n > PP_KPATH_MAX_N) return PP_ERR_LIMIT;
    const int m = n_cuts + 1;
    for (int j = 0; j < m; ++j) nodes[j] = -1;
    if (cut_threshold)
        for (int j = 0; j < n_cuts; ++j) cut_threshold[j] = 0;
    if (n_cuts == 0) {
        nodes[0] = 0;
        return PP_OK;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    try {
        // classes of the sizes by rank among the distinct values, highest class served first
        std::vector<uint64_t> distinct(sizes, sizes + n_cuts);
        std::sort(distinct.begin(), distinct.end());
        distinct.erase(std::unique(distinct.begin(), distinct.end()), distinct.end());
        std::vector<int> cls(n_cuts);
        for (int j = 0; j < n_cuts; ++j) {
            const size_t rank = std::lower_bound(distinct.begin(), distinct.end(), sizes[j]) - distinct.begin();
            cls[j] = (int)(rank * (size_t)n_classes / distinct.size());
        }
        // link bandwidths in descending order: the thresholds Algorithm 2 bisects over
        std::vector<uint32_t> edge_list;
        for (int v = 0; v < n; ++v)
            for (int w = 0; w < n; ++w)
                if (v != w && bw_kbps[v * n + w] > 0) edge_list.push_back(bw_kbps[v * n + w]);
        std::sort(edge_list.begin(), edge_list.end(), std::greater<uint32_t>());
        // device buffers for one batch of queries (the longest path decides their size)
        const size_t T = (size_t)trials;
        const size_t sz[8] = {(size_t)n * n * 4, T * 4, T * 4, T * 4, T * 8, T * n, T, T * PP_KPATH_MAX_K * 4};
        size_t off[9];
        off[0] = 0;
        for (int i = 0; i < 8; ++i) off[i + 1] = align_up(off[i] + sz[i], 256);
        unsigned char *buf = nullptr;
        PP_CUDA(staging_alloc(reinterpret_cast<void **>(&buf), off[8], s));
        struct Release {
            unsigned char *b; cudaStream_t st;
            ~Release() { cudaFreeAsync(b, st); cudaStreamSynchronize(st); }
        } release{buf, s};
        PP_CUDA(cudaMemcpyAsync(buf + off[0], bw_kbps, sz[0], cudaMemcpyHostToDevice, s));
        std::vector<uint32_t> h_thr(T);
        std::vector<int32_t> h_start(T), h_end(T), h_path(T * PP_KPATH_MAX_K);
        std::vector<uint64_t> h_alive(T);
        std::vector<uint8_t> h_col(T * n), h_found(T);
        uint64_t used = 0;
        for (int X = n_classes - 1; X >= 0; --X) {
            // maximal runs of cuts of class X, longest first, equal lengths by first cut
            std::vector<std::pair<int, int>> runs;  // (first cut, cuts)
            for (int i = 0; i < n_cuts;) {
                if (cls[i] != X) { ++i; continue; }
                int j = i;
                while (j < n_cuts && cls[j] == X) ++j;
                runs.emplace_back(i, j - i);
                i = j;
            }
            std::stable_sort(runs.begin(), runs.end(),
                             [](const std::pair<int, int> &a, const std::pair<int, int> &b) { return a.second > b.second; });
            for (const auto &run : runs) {
                const int first = run.first, cuts = run.second, kk = cuts + 1;
                if (kk > PP_KPATH_MAX_K) return PP_ERR_LIMIT;
                const int sv = nodes[first], uv = nodes[first + cuts];
                uint64_t alive = ~used;
                if (sv >= 0) alive |= 1ull << sv;
                if (uv >= 0) alive |= 1ull << uv;
                for (size_t t = 0; t < T; ++t) {
                    h_start[t] = sv;
                    h_end[t] = uv;
                    h_alive[t] = alive;
                    for (int v = 0; v < n; ++v)
                        h_col[t * n + v] = (uint8_t)(((uint64_t)draws[t * n + v] * (uint64_t)kk) >> 32);
                }
                PP_CUDA(cudaMemcpyAsync(buf + off[2], h_start.data(), sz[2], cudaMemcpyHostToDevice, s));
                PP_CUDA(cudaMemcpyAsync(buf + off[3], h_end.data(), sz[3], cudaMemcpyHostToDevice, s));
                PP_CUDA(cudaMemcpyAsync(buf + off[4], h_alive.data(), sz[4], cudaMemcpyHostToDevice, s));
                PP_CUDA(cudaMemcpyAsync(buf + off[5], h_col.data(), sz[5], cudaMemcpyHostToDevice, s));
                size_t low = 0, high = edge_list.size();
                std::vector<int32_t> best_path;
                uint32_t best_t = 0;
                while (low < high) {
                    const size_t median = (low + high) / 2;
                    std::fill(h_thr.begin(), h_thr.end(), edge_list[median]);
                    PP_CUDA(cudaMemcpyAsync(buf + off[1], h_thr.data(), sz[1], cudaMemcpyHostToDevice, s));
                    PP_CUDA(launch_kpath(n, kk, (int64_t)T, reinterpret_cast<uint32_t *>(buf + off[0]),
                                         reinterpret_cast<uint32_t *>(buf + off[1]), reinterpret_cast<int32_t *>(buf + off[2]),
                                         reinterpret_cast<int32_t *>(buf + off[3]),
                                         reinterpret_cast<unsigned long long *>(buf + off[4]), buf + off[5], buf + off[6],
                                         reinterpret_cast<int32_t *>(buf + off[7]), s));
                    PP_CUDA(cudaMemcpyAsync(h_found.data(), buf + off[6], T, cudaMemcpyDeviceToHost, s));
                    PP_CUDA(cudaMemcpyAsync(h_path.data(), buf + off[7], T * kk * 4, cudaMemcpyDeviceToHost, s));
                    PP_CUDA(cudaStreamSynchronize(s));
                    size_t hit = T;
                    for (size_t t = 0; t < T && hit == T; ++t)
                        if (h_found[t]) hit = t;  // the first colouring that finds a path
                    if (hit == T) {
                        low = median + 1;
                    } else {
                        high = median;
                        best_path.assign(h_path.begin() + hit * kk, h_path.begin() + (hit + 1) * kk);
                        best_t = edge_list[median];
                    }
                }
                if (best_path.empty()) {
                    for (int j = 0; j < m; ++j) nodes[j] = -1;
                    return PP_INFEASIBLE;
                }
                for (int i = 0; i < kk; ++i) {
                    nodes[first + i] = best_path[i];
                    used |= 1ull << best_path[i];
                }
                if (cut_threshold)
                    for (int i = 0; i < cuts; ++i) cut_threshold[first + i] = best_t;
            }
        }
    } catch (const std::bad_alloc &) {
        return PP_ERR_NOMEM;
    }
    return PP_OK;
}

pp_status pp_solve_exact_compute(int32_t L, const uint64_t *layer_out_bits, const uint64_t *layer_mem_bytes,
                                 const uint64_t *layer_work, int32_t k, const uint64_t *node_mem_bytes,
                                 const uint32_t *bw_kbps, const uint32_t *node_speed, double *beta_ms, int32_t *m,
                                 int32_t *cuts, int32_t *placement)
{
    if (!beta_ms || !m || !placement || (!cuts && k > 1) || !layer_work || !node_speed) return PP_ERR_ARG;
    pp_status st = validate(L, layer_out_bits, layer_mem_bytes, k, node_mem_bytes, bw_kbps);
    if (st != PP_OK) return st;
    if (L > PP_COMPUTE_MAX_L || k > PP_COMPUTE_MAX_K) return PP_ERR_LIMIT;
    for (int i = 0; i < L; ++i)
        if (layer_work[i] >= PP_MAX_BITS) return PP_ERR_LIMIT;
    try {
        std::vector<uint64_t> M(L + 1, 0), Wp(L + 1, 0);
        for (int i = 0; i < L; ++i) {
            M[i + 1] = M[i] + layer_mem_bytes[i];
            Wp[i + 1] = Wp[i] + layer_work[i];
        }
        DeviceMasks dmasks;
        PP_CUDA(device_masks(k, mask_list(k), &dmasks));
        struct Part { const void *src; size_t bytes; size_t off; };
        std::vector<Part> parts = {
            {layer_out_bits, (size_t)L * 8, 0}, {M.data(), (size_t)(L + 1) * 8, 0}, {Wp.data(), (size_t)(L + 1) * 8, 0},
            {node_mem_bytes, (size_t)k * 8, 0}, {bw_kbps, (size_t)k * k * 4, 0}, {node_speed, (size_t)k * 4, 0},
            {nullptr, 16, 0} /* best value, best key */, {nullptr, sizeof(pp_solution), 0},
            {nullptr, (size_t)k * k * L * 8, 0} /* gamma */, {nullptr, (size_t)k * L * L * 8, 0} /* compute times */,
            {nullptr, ((size_t)k << k) * L * 8, 0} /* state table */};
        size_t total = 0;
        for (auto &q : parts) { q.off = total; total = align_up(total + q.bytes, 256); }
        unsigned char *buf = nullptr;
        if (alloc_should_fail()) return PP_ERR_NOMEM;
        PP_CUDA(cudaMalloc(reinterpret_cast<void **>(&buf), total));
        struct Release {
            unsigned char *b;
            ~Release() { cudaFree(b); }
        } release{buf};
        cudaStream_t s = nullptr;
        for (int i = 0; i < 6; ++i)
            PP_CUDA(cudaMemcpyAsync(buf + parts[i].off, parts[i].src, parts[i].bytes, cudaMemcpyHostToDevice, s));
        CtDev d{};
        d.L = L; d.k = k;
        d.bits = reinterpret_cast<uint64_t *>(buf + parts[0].off);
        d.M = reinterpret_cast<uint64_t *>(buf + parts[1].off);
        d.Wp = reinterpret_cast<uint64_t *>(buf + parts[2].off);
        d.cap = reinterpret_cast<uint64_t *>(buf + parts[3].off);
        d.bw = reinterpret_cast<uint32_t *>(buf + parts[4].off);
        d.speed = reinterpret_cast<uint32_t *>(buf + parts[5].off);
        d.masks = dmasks.masks;
        d.level_off = dmasks.level_off;
        d.best_val = reinterpret_cast<unsigned long long *>(buf + parts[6].off);
        d.best_key = d.best_val + 1;
        pp_solution *d_sol = reinterpret_cast<pp_solution *>(buf + parts[7].off);
        d.gam = reinterpret_cast<double *>(buf + parts[8].off);
        d.seg = reinterpret_cast<double *>(buf + parts[9].off);
        d.table = reinterpret_cast<double *>(buf + parts[10].off);
        PP_CUDA(launch_compute_search(d, d_sol, s));
        pp_solution h{};
        PP_CUDA(cudaMemcpyAsync(&h, d_sol, sizeof h, cudaMemcpyDeviceToHost, s));
        PP_CUDA(cudaStreamSynchronize(s));
        if (h.status != PP_OK && h.status != PP_INFEASIBLE) return PP_ERR_CUDA;
        *beta_ms = h.beta_ms;
        *m = h.m;
        for (int j = 0; j < k - 1; ++j) cuts[j] = h.cuts[j];
        for (int j = 0; j < k; ++j) placement[j] = h.placement[j];
        return static_cast<pp_status>(h.status);
    } catch (const std::bad_alloc &) {
        return PP_ERR_NOMEM;
    }
}

pp_status pp_debug_minmax_rate(int32_t op, int32_t iters, double *warp_instr_per_clk_per_sm)
{
    if (!warp_instr_per_clk_per_sm || op < 0 || op > 2 || iters < 1 || iters > (1 << 20)) return PP_ERR_ARG;
    int dev = 0, sms = 0;
    PP_CUDA(cudaGetDevice(&dev));
    PP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned char *buf = nullptr;
    PP_CUDA(cudaMalloc(reinterpret_cast<void **>(&buf), (size_t)sms * 8 + 256));
    long long *cycles = reinterpret_cast<long long *>(buf);
    uint32_t *sink = reinterpret_cast<uint32_t *>(buf + (size_t)sms * 8);
    std::vector<long long> h;
    cudaError_t e = cudaSuccess;
    try {
        h.resize(sms);
    } catch (const std::bad_alloc &) {
        cudaFree(buf);
        return PP_ERR_NOMEM;
    }
    for (int rep = 0; rep < 3 && e == cudaSuccess; ++rep) e = launch_probe(op, iters, sms, cycles, sink, nullptr);
    if (e == cudaSuccess) e = cudaMemcpy(h.data(), cycles, (size_t)sms * 8, cudaMemcpyDeviceToHost);
    cudaFree(buf);
    if (e != cudaSuccess) return from_cuda(e);
    std::sort(h.begin(), h.end());
    const long long med = h[sms / 2];
    if (med <= 0) return PP_ERR_CUDA;
    *warp_instr_per_clk_per_sm = probe_instr_per_block(iters) / (double)med;
    return PP_OK;
}

pp_status pp_debug_fail_alloc(int32_t nth)
{
    if (nth < 0) return PP_ERR_ARG;
    g_fail_alloc_countdown.store(nth);
    return PP_OK;
}

pp_status pp_debug_mask_order(int32_t k, uint32_t *masks_out, uint32_t *level_off_out)
{
    if (!masks_out || !level_off_out || k < 1) return PP_ERR_ARG;
    if (k > PP_MAX_K) return PP_ERR_LIMIT;
    try {
        const MaskList &ml = mask_list(k);
        std::copy(ml.masks.begin(), ml.masks.end(), masks_out);
        std::copy(ml.level_off.begin(), ml.level_off.end(), level_off_out);
    } catch (const std::bad_alloc &) {
        return PP_ERR_NOMEM;
    }
    return PP_OK;
}

pp_status pp_debug_read_state_row(pp_problem *p, uint32_t mask, int32_t v, double *row_out)
{
    if (!p || !row_out || !p->solved) return PP_ERR_ARG;
    if (v < 0 || v >= p->k || mask >= (1u << p->k) || !((mask >> v) & 1u)) return PP_ERR_ARG;
    PP_CUDA(cudaStreamSynchronize(p->stream));
    const int L = p->L, U = p->U;
    std::vector<uint32_t> rk((size_t)std::max(U, 1) * L);
    std::vector<double> gu((size_t)std::max(U, 1) * L);
    if (U > 0) {
        PP_CUDA(cudaMemcpy(rk.data(), p->d.rk, (size_t)U * L * 4, cudaMemcpyDeviceToHost));
        PP_CUDA(cudaMemcpy(gu.data(), p->d.gu, (size_t)U * L * 8, cudaMemcpyDeviceToHost));
    }
    std::map<uint32_t, double> val;
    for (size_t i = 0; i < (size_t)U * L; ++i) val[rk[i]] = gu[i];
    const size_t row = ((size_t)mask * p->k + v) * p->Lpad;
    std::vector<uint32_t> raw(L);
    if (p->elem == 2) {
        std::vector<uint16_t> r16(L);
        PP_CUDA(cudaMemcpy(r16.data(), static_cast<uint16_t *>(p->d.table) + row, (size_t)L * 2,
                           cudaMemcpyDeviceToHost));
        for (int c = 0; c < L; ++c) raw[c] = r16[c] == 0xFFFFu ? 0xFFFFFFFFu : r16[c];
    } else {
        PP_CUDA(cudaMemcpy(raw.data(), static_cast<uint32_t *>(p->d.table) + row, (size_t)L * 4,
                           cudaMemcpyDeviceToHost));
    }
    for (int c = 0; c < L; ++c) {
        if (raw[c] == 0) row_out[c] = 0.0;
        else if (raw[c] == 0xFFFFFFFFu) row_out[c] = std::numeric_limits<double>::infinity();
        else {
            auto it = val.find(raw[c]);
            if (it == val.end()) return PP_ERR_CUDA;
            row_out[c] = it->second;
        }
    }
    return PP_OK;
}

}  // extern "C"
