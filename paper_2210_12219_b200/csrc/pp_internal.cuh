// Internal declarations shared by the translation units of libpp (host launchers + device view).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "pp.h"

namespace pp {

// Device view of one problem.  Ranks are an order-preserving recoding of the gamma doubles:
// 0 stands for +0.0, the all-ones value of the element type for +inf, 1..N for the gamma
// values in increasing order (equal doubles share a rank).  min/max/compare on ranks give the
// same selections as on the doubles (the sweep never does arithmetic on values).
struct Dev {
    int L, k, Lpad;            // Lpad: row stride in elements (32-byte multiple)
    int U;                     // number of distinct non-zero off-diagonal bandwidth values
    int elem;                  // bytes per state element: 2 or 4
    const uint64_t *bits;      // [L]
    const uint64_t *M;         // [L+1] prefix sums of layer memory
    const uint64_t *cap;       // [k]
    const uint32_t *bw;        // [k*k]
    const int16_t *lo;         // [k*L] lo[w*L+c'] = first c >= 0 whose successor segment c+1..c' fits w
                               //        (= c' when even the single layer c' does not fit)
    const int16_t *pair_u;     // [k*k] index into ubw of the pair's bandwidth, -1 if unusable
    const uint32_t *ubw;       // [U] distinct bandwidth values
    const uint32_t *masks;     // [2^k - 1] all non-empty masks by popcount, each level in revolving-door
                               //        order (neighbours differ by one node swapped for another)
    const uint32_t *level_off; // [k+2] masks of popcount j are masks[level_off[j] .. level_off[j+1])
    int16_t *pos;              // [L] position of layer c in the ascending order of bits
    int16_t *order;            // [L] layer at each position
    double *gu;                // [U*L] gu[u*L+i] = bits[order[i]] / ubw[u]  (ascending in i)
    uint32_t *cnt;             // [U*L] number of quotients below gu[u*L+i] (accumulated by the rank build)
    uint32_t *rk;              // [U*L] rank of gu[u*L+i] = 1 + cnt
    uint32_t *inv;             // [U*L+2] inv[r] = some entry e with rk[e] == r (equal ranks hold equal doubles)
    void *rank;                // [k*k*Lpad] rank[(w*k+v)*Lpad + c] of gamma[c][v][w], element type
    void *table;               // [2^k * k * Lpad] state rows, row (S, v) at (S*k+v)*Lpad
    uint64_t table_elems;      // elements of the state table / of the rank table: what an index
    uint64_t rank_elems;       //        may reach (checked only in the bounds-checking build)
    unsigned long long *best;  // packed (rank, popcount, mask, v) of the best final state
    int32_t *err;              // device error word (0 = fine, kErrBacktrack)
    const void *fast_meta;     // per-node window constants of the register-tiled sweep, or null
    const uint32_t *gen_meta;  // [k*Lpad] per-(node, position) lookup words of its general-window step, or null
    int gen_levels;            // levels of that step's sparse table (1 + floor(log2(longest window)))
    const void *pair_meta;     // per-node window constants of the two-mask sweep, or null
};

static constexpr unsigned long long kNoBest = ~0ull;
static constexpr int32_t kErrBacktrack = 1;  // the backtrack found no predecessor (inconsistent table)
static constexpr int32_t kErrBounds = 3;     // bounds-checking build: an index left its table

// Bounds-checking build (-DPP_DEBUG_BOUNDS, libpp_dbg.so): every access to the state table and to
// the rank table in global memory goes through PP_IN_BOUNDS, which records kErrBounds in the
// device error word and makes the caller skip the access when the index is outside the table.
// Nothing traps; the solve then returns PP_ERR_CUDA.  In the normal build the check is `true`.
#ifdef PP_DEBUG_BOUNDS
#define PP_IN_BOUNDS(d, index, limit) \
    ((uint64_t)(index) < (uint64_t)(limit) ? true : (atomicCAS((d).err, 0, kErrBounds), false))
#else
#define PP_IN_BOUNDS(d, index, limit) true
#endif

// final-state key: smaller is better; rank in the high bits, then popcount, mask, node
__host__ __device__ inline unsigned long long pack_best(uint32_t rank, int popc, uint32_t mask, int v)
{
    return ((unsigned long long)rank << 30) | ((unsigned long long)popc << 25) |
           ((unsigned long long)mask << 5) | (unsigned long long)v;
}

cudaError_t launch_rank_base(const Dev &d, cudaStream_t s, int *launches);
cudaError_t launch_sweep_generic(const Dev &d, int level, cudaStream_t s);
size_t fast_meta_bytes();
bool fast_meta_build(int L, int k, const int16_t *lo, void *out);
int gen_meta_build(int L, int k, int Lpad, const int16_t *lo, uint32_t *out);
bool fast_sweep_supported(const Dev &d);
// first_level: the kernel follows the rank build directly and must wait for it before reading anything
cudaError_t launch_sweep_fast(const Dev &d, int level, cudaStream_t s, bool first_level);
size_t pair_meta_bytes();
bool pair_meta_build(int L, int k, const int16_t *lo, void *out);
bool pair_sweep_takes(const Dev &d, int level, bool whenever_possible);
cudaError_t launch_sweep_pair(const Dev &d, int level, cudaStream_t s, bool first_level);
cudaError_t launch_finalize(const Dev &d, pp_solution *out, cudaStream_t s, bool dependent);
cudaError_t launch_eval(const Dev &d, int64_t B, const uint8_t *nseg, const int32_t *ends,
                        const int32_t *nodes, double *beta, uint8_t *status, cudaStream_t s);
cudaError_t launch_eval_packed(const Dev &d, int64_t B, int64_t total, const uint8_t *nseg, const uint32_t *off,
                               const uint16_t *ends, const uint8_t *nodes, double *beta, uint8_t *status,
                               cudaStream_t s);
size_t batch_smem_bytes(int L, int k);
cudaError_t launch_batch(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                         const uint64_t *cap, const uint32_t *bw, double *beta, int32_t *m,
                         int32_t *cuts, int32_t *placement, int8_t *status, cudaStream_t s);
// Many-instance search with one instance per lane (pp_batch_lanes.cu): tables of a chunk of
// instances in global memory, instance-minor, so that the 32 lanes of a warp read 32 neighbouring
// words.  Group g holds instances 32 g .. 32 g + 31 of the chunk.
struct BatchLanes {
    uint32_t *table;          // [group][compact row][LH][32]: states, two cut positions per word
    uint32_t *rank;           // [group][v * k + w][LH][32]: gamma ranks, same packing
    uint32_t *len;            // [group][w][LH][32]: window lengths c' - lo_w(c'), same packing
    uint32_t *win;            // [group][w][2 LH][32]: per cut position the two sparse-table cells whose minimum
                              // is the window minimum, as byte offsets into a warp's table (see pp_batch_lanes.cu)
    unsigned long long *key;  // [group][32]: smallest final state so far (value, popcount, mask, node)
    int8_t *flag;             // [group][32]: 1 = an input beyond the limits
    int32_t *err;             // device error word (bounds-checking build: kErrBounds when an index left its table)
    size_t table_words, rank_words, len_words, win_words;  // sizes of the four tables in 32-bit words
    const uint32_t *rowoff;   // [2^k]: compact row of (S, lowest node of S), rows ordered by (popcount, mask, node)
    const uint32_t *mlist;    // masks by (popcount, value)
    const uint32_t *moff;     // [k + 2]: first entry of each popcount in mlist
    uint32_t rows;            // k * 2^(k-1)
    int LH;                   // words per row in these tables: 4, 8, 12 or 16
};
bool batch_lanes_takes(int64_t B, int L, int k);
int batch_lanes_words(int L);
// prep: one warp per instance ranks gamma and writes the instance's column of the tables
cudaError_t launch_batch_prep(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                              const uint64_t *cap, const uint32_t *bw, const BatchLanes &t, cudaStream_t s);
// the levels and the backtrack over a prepared chunk; *launches counts the kernels queued
cudaError_t launch_batch_lanes(int64_t B, int L, int k, const uint64_t *bits, const uint32_t *bw,
                               const BatchLanes &t, double *beta, int32_t *m, int32_t *cuts,
                               int32_t *placement, int8_t *status, cudaStream_t s);
// Random comparison baseline (Section 4): P plans of problem d from 2 k draws each.
cudaError_t launch_random_plans(const Dev &d, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                                int32_t *nodes, cudaStream_t s);
// Greedy comparison baseline (Section 4), one warp per instance.
cudaError_t launch_greedy(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                          const uint64_t *cap, const uint32_t *bw, double *beta, int32_t *m, int32_t *cuts,
                          int32_t *place, int8_t *status, cudaStream_t s);

// Partition stage of the paper's heuristic (Algorithm 1), one warp per chain.
size_t partition_smem_bytes(int L);
cudaError_t launch_partition_minsum(int64_t B, int L, int cap_seg, const uint64_t *weight, const uint64_t *mem,
                                    const uint64_t *kappa, uint64_t *cost, int32_t *m, int32_t *cuts,
                                    uint64_t *sizes, int8_t *status, cudaStream_t s);
// Colour-coding k-path search of the placement stage (Algorithm 2's K-PATH), one block per query.
size_t kpath_smem_bytes(int kk);
cudaError_t launch_kpath(int n, int kk, int64_t Q, const uint32_t *bw, const uint32_t *threshold, const int32_t *start,
                         const int32_t *end, const unsigned long long *alive, const uint8_t *colours, uint8_t *found,
                         int32_t *path, cudaStream_t s);
// Exact search under Eq. 1 (compute times in the bottleneck), pp_compute.cu.
struct CtDev {
    int L, k;
    const uint64_t *bits, *M, *Wp, *cap;   // [L], [L+1] memory prefix sums, [L+1] work prefix sums, [k]
    const uint32_t *bw, *speed;            // [k*k], [k]
    const uint32_t *masks, *level_off;     // node sets by popcount (any order within a level)
    double *gam, *seg, *table;             // [k*k*L], [k*L*L], [2^k * k * L]
    unsigned long long *best_val, *best_key;  // adjacent 64-bit words
};
cudaError_t launch_compute_search(const CtDev &d, pp_solution *out, cudaStream_t s);
// Issue-rate probe (pp_probe.cu): `blocks` blocks of 1024 threads, cycles[b] = SM clocks block b took.
cudaError_t launch_probe(int op, int iters, int blocks, long long *cycles, uint32_t *sink, cudaStream_t s);
double probe_instr_per_block(int iters);

}  // namespace pp
