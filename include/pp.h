/*
 * pp.h -- exact min-bottleneck partition-and-placement on one NVIDIA B200 (sm_100a).
 *
 * Problem (paper, Section 1 and Section 3.2).  A chain of L layers is cut into m >= 1
 * contiguous non-empty segments; segment j runs on its own edge node n_j, all nodes
 * different; a segment fits when the bytes of its layers are <= the node's capacity.  The
 * tensor that crosses cut j is the output of the last layer of segment j; its latency is
 *        gamma_j = bits[e_j] / bw[n_j][n_{j+1}]            (Eq. 3, data / bandwidth)
 * and a plan's bottleneck latency is
 *        beta = max_j gamma_j                              (Eq. 2),   beta = +0.0 if m = 1.
 * The library finds beta* = min over all plans, returns one canonical optimal plan, and
 * scores arbitrary candidate plans in bulk.
 *
 * Arithmetic contract.  gamma is ONE IEEE-754 binary64 round-to-nearest division of the
 * integer bit count by the integer kbps, so beta is in milliseconds.  The search only
 * compares and selects gamma values (min / max); beta* is bit-for-bit one of them, or +0.0,
 * or +inf.  A link of 0 kbps is unusable (gamma = +inf); the diagonal of bw is ignored.
 *
 * Canonical plan.  Among all plans with beta == beta*, the lexicographically smallest key
 *        (m, mask, n_m, e_{m-1}, n_{m-1}, ..., e_1, n_1),   mask = sum_j 2^{n_j}:
 * fewest segments, then lowest node-set mask, then lowest last node, then, walking
 * backwards, lowest cut and lowest node id.
 *
 * Conventions for every entry point:
 *  - "host" / "device" on a pointer says where the memory must live.  The library never
 *    frees or keeps caller memory; inputs of pp_problem_create are copied.
 *  - Errors are return codes only.  On PP_ERR_* the outputs are untouched.
 *  - All work of a problem runs on its CUDA stream (default: the legacy default stream).
 *    The *_dev entry points are asynchronous on that stream; the host entry points
 *    synchronise it before returning.
 *  - Layers are 0..L-1, nodes 0..k-1.  A cut value e means "the segment ends with layer e".
 *  - There is no CPU fallback: without a CUDA device every compute entry point fails with
 *    PP_ERR_CUDA.
 */
#ifndef PP_H
#define PP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PP_MAX_K 20   /* nodes; the state table has k * 2^k rows */
#define PP_MAX_L 1024 /* layers */
#define PP_MAX_BITS (1ull << 40) /* layer_out_bits must be below this */
#define PP_MAX_KBPS (1u << 24)   /* bw_kbps must be below this */

typedef struct pp_problem pp_problem; /* opaque; owns host and device copies of the inputs */

typedef enum {
    PP_OK = 0,
    PP_INFEASIBLE = 1, /* not an error: no plan exists; beta = +inf, m = 0 */
    PP_ERR_ARG = -1,   /* null pointer, L < 1, k < 1, B < 0 */
    PP_ERR_LIMIT = -2, /* k > PP_MAX_K, L > PP_MAX_L, value above PP_MAX_BITS / PP_MAX_KBPS,
                          or (batched solve) a shape whose tables do not fit shared memory */
    PP_ERR_NOMEM = -3, /* host or device allocation failed, or workspace too small */
    PP_ERR_CUDA = -4,  /* a CUDA runtime call failed (includes "no device") */
    PP_ERR_TIMEOUT = -5 /* reserved */
} pp_status;

/* plan_status bit flags written by the evaluator (0 = valid plan) */
#define PP_PLAN_BAD_NSEG 1   /* nseg == 0 or nseg > min(k, L); nothing else is checked */
#define PP_PLAN_BAD_ENDS 2   /* a cut outside [0, L-2] or cuts not strictly increasing */
#define PP_PLAN_BAD_NODE 4   /* a node outside [0, k-1] or used twice */
#define PP_PLAN_MEMORY 8     /* some segment exceeds its node's capacity */
#define PP_PLAN_DEAD_LINK 16 /* two consecutive nodes joined by a 0 kbps link */

/* Result record of the exact search as the device writes it. */
typedef struct {
    double beta_ms;              /* beta*, +inf if infeasible */
    int32_t status;              /* PP_OK or PP_INFEASIBLE; PP_ERR_CUDA when the backtrack broke off */
    int32_t m;                   /* number of segments, 0 if infeasible */
    int32_t cuts[PP_MAX_K];      /* e_1 .. e_{m-1}; unused slots are -1 */
    int32_t placement[PP_MAX_K]; /* n_1 .. n_m;     unused slots are -1 */
} pp_solution;

/* Device-time breakdown of the last pp_solve_exact / pp_solve_exact_dev of a problem. */
typedef struct {
    float ms_rank;     /* gamma table, rank compression (Eq. 3) and the base frontier (one node used) */
    float ms_sweep;    /* all popcount levels (two nodes and more) of the (min,max) sweep */
    float ms_finalize; /* final choice and backtrack */
    float ms_total;
    int32_t sweep_launches;  /* kernels launched for the sweep: one per popcount level from 2 up */
    int32_t total_launches;  /* all kernels of the solve */
    int32_t state_bytes;     /* bytes of one state element: 2 (16-bit ranks) or 4 */
    int32_t fast_path;       /* register-tiled sweep: 1 = constant-width windows, 2 = general
                                windows; 0 = the generic kernel ran */
    int32_t pair_levels;     /* popcount levels swept by the kernel that takes two source masks
                                per warp (constant-width windows only) */
} pp_profile;

/*
 * Problem set-up (Section 3: inputs are the chain and the weighted communication graph).
 *   layer_out_bits  host [L]    output size of each layer in bits (transfer size of a cut after it)
 *   layer_mem_bytes host [L]    memory of each layer in bytes
 *   node_mem_bytes  host [k]    capacity of each node in bytes (heterogeneous; the paper's
 *                               homogeneous case is all entries equal)
 *   bw_kbps         host [k*k]  row-major, [v*k + w] = bandwidth of the link v -> w; 0 = no link
 * Validates, builds the uint64 memory prefix sums and the per-node window table (for each
 * node w and segment end c', the earliest segment start that still fits), uploads them.
 * *out receives the handle; free it with pp_problem_destroy.
 * The list of node sets the search walks depends on k only: its device copy (4 * 2^k bytes) is
 * made by the first problem of that k on a device and kept until the process ends.
 */
pp_status pp_problem_create(int32_t L, const uint64_t *layer_out_bits,
                            const uint64_t *layer_mem_bytes, int32_t k,
                            const uint64_t *node_mem_bytes, const uint32_t *bw_kbps,
                            pp_problem **out);

/* Frees the handle and every device buffer the library allocated for it (not a caller
 * workspace).  NULL is allowed. */
void pp_problem_destroy(pp_problem *p);

/* Use `cuda_stream` (a cudaStream_t, e.g. torch.cuda.current_stream().cuda_stream) for all
 * later work of this problem.  NULL selects the legacy default stream. */
pp_status pp_problem_set_stream(pp_problem *p, void *cuda_stream);

/* Bytes of device scratch the exact search needs (state table, gamma and rank tables). */
pp_status pp_problem_workspace_bytes(const pp_problem *p, uint64_t *bytes);

/* Hand the library a caller-owned device buffer (256-byte aligned, at least
 * pp_problem_workspace_bytes) to use instead of allocating its own at the first solve.
 * The caller keeps ownership and must keep it alive while the problem is used. */
pp_status pp_problem_set_workspace(pp_problem *p, void *device_buffer, uint64_t bytes);

/*
 * Exact search (Eq. 2 minimised over every cut set and every injective placement) by a
 * (min,max) dynamic programme over (used-node mask, last node, last cut layer), swept by
 * popcount of the mask; then the canonical plan by backtracking.
 *   beta_ms   host [1]    beta* in milliseconds, +inf if infeasible
 *   m         host [1]    number of segments, 0 if infeasible
 *   cuts      host [k-1]  e_1..e_{m-1}, rest -1   (may be NULL when k == 1)
 *   placement host [k]    n_1..n_m, rest -1
 * Returns PP_OK, PP_INFEASIBLE or an error.  Synchronous.
 */
pp_status pp_solve_exact(pp_problem *p, double *beta_ms, int32_t *m, int32_t *cuts,
                         int32_t *placement);

/* Same search; the result record is written to device memory `solution_dev` (device,
 * sizeof(pp_solution), 8-byte aligned) by work queued on the problem's stream.  Returns as
 * soon as the work is queued; feasibility is in solution_dev->status. */
pp_status pp_solve_exact_dev(pp_problem *p, pp_solution *solution_dev);

/*
 * Batched beta evaluator (Eq. 3 per cut, Eq. 2 per plan) for B candidate plans of one problem.
 *   nseg        [B]    number of segments of each plan
 *   ends        [B*k]  row b: cuts e_1..e_{nseg-1} (only the first nseg-1 entries are read;
 *                      the last segment always ends at L-1)
 *   nodes       [B*k]  row b: n_1..n_nseg (only the first nseg entries are read)
 *   beta_ms     [B]    out: beta of the plan, +inf if any flag is set
 *   plan_status [B]    out: PP_PLAN_* flags.  BAD_NSEG stops all other checks; MEMORY and
 *                      DEAD_LINK are only evaluated when ENDS and NODE are clean.
 * pp_eval_plans takes host pointers and is synchronous; pp_eval_plans_dev takes device
 * pointers and is asynchronous on the problem's stream.  B == 0 is a no-op.
 */
pp_status pp_eval_plans(pp_problem *p, int64_t B, const uint8_t *nseg, const int32_t *ends,
                        const int32_t *nodes, double *beta_ms, uint8_t *plan_status);
pp_status pp_eval_plans_dev(pp_problem *p, int64_t B, const uint8_t *nseg, const int32_t *ends,
                            const int32_t *nodes, double *beta_ms, uint8_t *plan_status);

/*
 * The same evaluator (Eq. 3 per cut, Eq. 2 per plan, same validity rules and flags) for plans in
 * compressed rows: a third of the bytes of the int32 layout, for callers that score plans in bulk.
 *   nseg      [B]      number of segments of each plan
 *   plan_off  [B + 1]  plan b owns entries plan_off[b] .. plan_off[b + 1] - 1 of `ends` and `nodes`
 *                      (non-decreasing; normally the running sum of nseg)
 *   ends      [total]  16-bit cuts: the first nseg - 1 entries of a plan's row are read
 *   nodes     [total]  8-bit node ids: the first nseg entries of a plan's row are read
 *   beta_ms [B], plan_status [B]   out, as for pp_eval_plans; a row that holds fewer than nseg
 *                      entries, or reaches beyond `total`, is flagged PP_PLAN_BAD_NSEG
 * Host variant: host pointers, synchronous.  _dev variant: device pointers, asynchronous on the
 * problem's stream.  B == 0 is a no-op.
 */
pp_status pp_eval_plans_packed(pp_problem *p, int64_t B, int64_t total, const uint8_t *nseg,
                               const uint32_t *plan_off, const uint16_t *ends, const uint8_t *nodes,
                               double *beta_ms, uint8_t *plan_status);
pp_status pp_eval_plans_packed_dev(pp_problem *p, int64_t B, int64_t total, const uint8_t *nseg,
                                   const uint32_t *plan_off, const uint16_t *ends, const uint8_t *nodes,
                                   double *beta_ms, uint8_t *plan_status);

/*
 * Many independent instances of the same shape (L, k) in one call; each instance is the
 * exact search above.
 *   out_bits [B*L], mem [B*L], node_mem [B*k], bw [B*k*k]   inputs, instance-major
 *   beta_ms [B], m [B], cuts [B*(k-1)], placement [B*k], status [B] (PP_OK / PP_INFEASIBLE,
 *   or PP_ERR_LIMIT for an instance with a value above the limits)
 * Two device paths give the same results.  From 64 instances on, with 2 <= k <= 8 and L <= 32, a
 * warp sweeps 32 instances at once (one per lane); the state, rank and window tables of up to 4096
 * instances at a time live in scratch memory that the call takes from the library's own memory pool
 * and gives back, both ordered on the stream (k = 8, L = 24: 53 KB per instance; PP_ERR_NOMEM if
 * the pool cannot supply it; longer batches are worked off in pieces of 4096 on the same stream).
 * Otherwise one thread block solves one instance with its whole state table in shared memory.
 * Returns PP_ERR_LIMIT without touching outputs when the instance shape does not fit one block:
 * k > 12, k*(k-1)*L + 1 > 65534 (ranks are 16-bit), or k * 2^(k-1) * L 16-bit states plus the
 * rank tables beyond the shared memory of a block (k = 8, L = 24 needs 73 KB).  Host variant is
 * synchronous and uses the legacy default stream; the _dev variant takes device pointers and a
 * stream and is asynchronous.  cuts may be NULL when k == 1.
 */
pp_status pp_solve_exact_batch(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                               const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                               double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement,
                               int8_t *status);
pp_status pp_solve_exact_batch_dev(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                                   const uint64_t *mem, const uint64_t *node_mem,
                                   const uint32_t *bw, double *beta_ms, int32_t *m, int32_t *cuts,
                                   int32_t *placement, int8_t *status, void *cuda_stream);

/*
 * Random comparison baseline of Section 4 (first algorithm of the paper's comparison list) as a
 * generator of P candidate plans of one problem, in the evaluator's input layout.  Step s of a
 * plan takes a random node among the nodes not used yet and a random segment among those that
 * start at the next unassigned layer and fit that node's memory, until the chain is used up.
 *   draws [P*2k]  32-bit random numbers supplied by the caller; row p, word 2s chooses the node of
 *                 step s, word 2s+1 its segment; a draw d picks index floor(d * n / 2^32) among n
 *                 candidates in ascending order (both choices uniform: the paper does not say)
 *   nseg [P], ends [P*k], nodes [P*k]   out: as pp_eval_plans reads them, unused entries -1;
 *                 nseg = 0 (a row the evaluator flags PP_PLAN_BAD_NSEG) when the chosen node holds
 *                 not even the next layer or when all k nodes are used and layers are left over
 * Bandwidths play no part; score the plans with pp_eval_plans.  pp_random_plans takes host
 * pointers and is synchronous; pp_random_plans_dev takes device pointers and is asynchronous on
 * the problem's stream.  P == 0 is a no-op.
 */
pp_status pp_random_plans(pp_problem *p, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                          int32_t *nodes);
pp_status pp_random_plans_dev(pp_problem *p, int64_t P, const uint32_t *draws, uint8_t *nseg,
                              int32_t *ends, int32_t *nodes);

/*
 * Greedy comparison baseline of Section 4 (second algorithm of the paper's comparison list), for
 * many independent instances of the same shape; arguments, layouts and outputs as for
 * pp_solve_exact_batch, any L <= PP_MAX_L and k <= PP_MAX_K.  A walk starts on one node and
 * repeats two choices until the chain is used up: on the current node, among the segments that
 * start at the next unassigned layer and fit the node's memory, it takes the one with the
 * smallest outgoing transfer; then it moves to the unused node behind the current node's fastest
 * outgoing link.  One walk is made per start node and the one with the smallest bottleneck
 * latency is returned (Eq. 2, Eq. 3).  Where the paper is silent: a segment that reaches the last
 * layer transfers nothing and is taken as soon as it fits; equal transfers take the longer
 * segment, equal links the lower node, equal bottlenecks the lower start node; bandwidth 0 is no
 * link.  Values are not range-checked here (no PP_ERR_LIMIT per instance): the walk compares
 * integers and divides once per cut, which is exact in the sense of Eq. 3 for bit counts below
 * 2^53.  status[b] is PP_OK, or PP_INFEASIBLE when every walk gets stuck (the
 * heuristic found no plan; the exact search may still find one); then beta_ms = +inf, m = 0 and
 * the plan rows are -1.  Host variant: synchronous, legacy default stream.  _dev variant: device
 * pointers, asynchronous on `cuda_stream`.  cuts may be NULL when k == 1.
 */
pp_status pp_greedy_batch(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                          const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                          double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement,
                          int8_t *status);
pp_status pp_greedy_batch_dev(int64_t B, int32_t L, int32_t k, const uint64_t *out_bits,
                              const uint64_t *mem, const uint64_t *node_mem, const uint32_t *bw,
                              double *beta_ms, int32_t *m, int32_t *cuts, int32_t *placement,
                              int8_t *status, void *cuda_stream);

/*
 * Partition stage of the paper's two-stage heuristic (Section 3.2.1: the partition graph of Eq. 6
 * and Eq. 7, Algorithm 1), for B independent chains of the same length: cut the chain into
 * contiguous partitions that each fit one node's memory kappa (the paper's homogeneous capacity),
 * so that the sum of the weights of the cuts is smallest.  A cut after point c weighs
 * cut_weight[c]: the paper uses the transfer-size class of the point, pass raw sizes or class
 * numbers.  Of several plans with the same sum the one with fewer partitions is returned, then the
 * one whose cuts come earlier (the paper leaves ties open).
 *   cut_weight [B*L], mem [B*L], kappa [B]     inputs, chain-major; weights below PP_MAX_BITS
 *   cap_seg    rows of `cuts` / `sizes` have this many entries (cuts beyond it are not written)
 *   cost [B]   sum of the weights of the chosen cuts;  m [B] number of partitions
 *   cuts [B*cap_seg]   Q: last point of every partition but the final one, rest -1
 *   sizes [B*cap_seg]  S: cut_weight at those points, rest 0 (may be NULL)
 *   status [B] PP_OK; PP_INFEASIBLE (some point exceeds kappa: cost 0, m 0); PP_ERR_LIMIT (a weight
 *              above the limit or a wrapping memory sum, or m - 1 > cap_seg: cost and m are still set)
 * The cuts feed pp_eval_plans as `ends` once nodes are chosen for the partitions.  Host variant:
 * host pointers, synchronous, legacy default stream.  _dev variant: device pointers, asynchronous
 * on `cuda_stream`.  B == 0 is a no-op.
 */
pp_status pp_partition_minsum_batch(int64_t B, int32_t L, const uint64_t *cut_weight, const uint64_t *mem,
                                    const uint64_t *kappa, int32_t cap_seg, uint64_t *cost, int32_t *m,
                                    int32_t *cuts, uint64_t *sizes, int8_t *status);
pp_status pp_partition_minsum_batch_dev(int64_t B, int32_t L, const uint64_t *cut_weight, const uint64_t *mem,
                                        const uint64_t *kappa, int32_t cap_seg, uint64_t *cost, int32_t *m,
                                        int32_t *cuts, uint64_t *sizes, int8_t *status, void *cuda_stream);

/*
 * Inner step of the paper's placement stage (Section 3.2.2): the threshold classifier of Eq. 8 and
 * the K-PATH call of Algorithm 2, i.e. the colour-coding search for a simple path of kk vertices in
 * the subgraph of class-X links, for Q queries on one communication graph.
 *   n, bw_kbps [n*n]   the communication graph, as for pp_problem_create (row = sender), n <= 64
 *   kk                 vertices of the path looked for (the paper's k), kk <= 13, same for all queries
 *   threshold [Q]      Eq. 8: a link is class X, and part of the searched subgraph, when its bandwidth
 *                      is >= threshold (0 kbps is never a link); Algorithm 2's binary search over the
 *                      sorted bandwidths is a sequence of such queries
 *   start, end [Q]     first / last vertex of the path, -1 = any (Algorithm 2's s and u); a walk that
 *                      reaches `end` before it has kk vertices is not continued
 *   alive [Q]          bit v set = node v is still available (Algorithm 2 deletes placed nodes)
 *   colours [Q*n]      colour of every node, below kk (a node with a colour >= kk is not used); the
 *                      random colouring of the method is the caller's draw, repeated over queries
 *   found [Q]          out: 1 when a path of kk vertices with kk different colours exists
 *   path [Q*kk]        out: one such path (any valid one), -1 when none
 * The paper calls the classifier twice in a row in Algorithm 2 (once with the median edge, once
 * with `threshold`); here one threshold per query is taken, the median edge's bandwidth.
 * Host variant: host pointers, synchronous, legacy default stream.  _dev variant: device pointers,
 * asynchronous on `cuda_stream`.  Q == 0 is a no-op.
 */
#define PP_KPATH_MAX_N 64
#define PP_KPATH_MAX_K 13
pp_status pp_kpath_colour_batch(int32_t n, const uint32_t *bw_kbps, int64_t Q, int32_t kk, const uint32_t *threshold,
                                const int32_t *start, const int32_t *end, const uint64_t *alive,
                                const uint8_t *colours, uint8_t *found, int32_t *path);
pp_status pp_kpath_colour_batch_dev(int32_t n, const uint32_t *bw_kbps, int64_t Q, int32_t kk,
                                    const uint32_t *threshold, const int32_t *start, const int32_t *end,
                                    const uint64_t *alive, const uint8_t *colours, uint8_t *found, int32_t *path,
                                    void *cuda_stream);

/*
 * Placement stage of the paper's two-stage heuristic (Section 3.2.2, Algorithm 2 SUBGRAPH-K-PATH and
 * Algorithm 3 K-PATH-MATCHING): nodes for the n_cuts + 1 partitions that the partition stage left,
 * cut j joining node j and node j + 1.  The cut sizes are put into n_classes classes by their rank
 * among the distinct sizes; classes are served from the highest down, within a class the maximal
 * runs of consecutive cuts longest first (equal lengths by first cut); a run of l cuts gets a path
 * of l + 1 unused nodes between its already placed neighbours, at the largest link-bandwidth
 * threshold (Eq. 8) for which the colour-coding search of pp_kpath_colour_batch finds one: the
 * bisection of Algorithm 2 over the sorted bandwidths, each probe a batch of `trials` colourings,
 * the first colouring that finds a path decides.
 *   n, bw_kbps [n*n]   host: the communication graph (row = sender), n <= 64
 *   n_cuts, sizes [n_cuts]   host: transfer sizes S of the cuts, in chain order
 *   n_classes          number of transfer-size (= bandwidth) classes, >= 1
 *   trials, draws [trials*n]  host: 32-bit random numbers of the caller; node v gets colour
 *                      floor(draw * k / 2^32) in a search for a path of k vertices
 *   nodes [n_cuts+1]   host out: N, all different; -1 when the stage fails
 *   cut_threshold [n_cuts]   host out, may be NULL: the threshold found for the run of each cut
 * Returns PP_OK; PP_INFEASIBLE when some run finds no path at any threshold (the paper then runs the
 * stage again with fewer classes: the caller's loop); PP_ERR_LIMIT for n > 64 or a run of more than
 * 12 cuts.  Where the paper's listings are inconsistent (the classifier called twice, the path length
 * taken from the list of runs, the end vertex read one past the run) the readings are those of the
 * description above.  Synchronous; the device work runs on `cuda_stream`.
 */
pp_status pp_kpath_matching(int32_t n, const uint32_t *bw_kbps, int32_t n_cuts, const uint64_t *sizes,
                            int32_t n_classes, int32_t trials, const uint32_t *draws, int32_t *nodes,
                            uint32_t *cut_threshold, void *cuda_stream);

/*
 * Exact search under the paper's full objective, Eq. 1: beta = max over the plan's partitions and
 * cuts of { c_k, gamma_k }, the compute time of every partition counted as well (Eq. 2, which
 * pp_solve_exact minimises, drops it: the paper argues that transfers dominate on its hardware).
 *   layer_work  host [L]  computation of each layer in work units (below PP_MAX_BITS)
 *   node_speed  host [k]  work units per millisecond of each node; 0 = the node cannot compute
 * c_k = (exact integer sum of the partition's work) / (speed of its node): one IEEE-754 binary64
 * division, in milliseconds, like gamma.  All other arguments, the constraints, the canonical plan
 * and the outputs are those of pp_problem_create + pp_solve_exact.  One call does everything
 * (allocates its tables, runs, frees); synchronous, legacy default stream.  The state table holds
 * doubles (k * 2^k * L * 8 bytes) and every compute time has its own table entry (k * L * L * 8
 * bytes): PP_ERR_LIMIT beyond k = 16 or L = 256, PP_ERR_NOMEM when the device cannot hold them.
 * With layer_work all zero the result is that of pp_solve_exact.
 */
#define PP_COMPUTE_MAX_K 16
#define PP_COMPUTE_MAX_L 256
pp_status pp_solve_exact_compute(int32_t L, const uint64_t *layer_out_bits, const uint64_t *layer_mem_bytes,
                                 const uint64_t *layer_work, int32_t k, const uint64_t *node_mem_bytes,
                                 const uint32_t *bw_kbps, const uint32_t *node_speed, double *beta_ms, int32_t *m,
                                 int32_t *cuts, int32_t *placement);

/* Device-time breakdown of the last exact solve of `p`; synchronises the problem's stream.
 * ms_total is always measured.  ms_rank, ms_sweep and ms_finalize need events between the
 * phases, which keep one phase's kernels from being launched under the tail of the previous
 * one: they are recorded only after pp_problem_set_profiling(p, 1) and read 0 otherwise. */
pp_status pp_last_solve_profile(pp_problem *p, pp_profile *out);
pp_status pp_problem_set_profiling(pp_problem *p, int32_t on);

/* Test hook: after a solve, copy one row of the state table to the host as latencies:
 * row_out[c] = value of state (mask, v, c) in milliseconds (+inf if unreachable), c = 0..L-1.
 * `mask` must contain node v.  Synchronous. */
pp_status pp_debug_read_state_row(pp_problem *p, uint32_t mask, int32_t v, double *row_out);

/* Test hook (host only, needs no device): the order in which the sweep lists the non-empty node
 * sets of k nodes.  masks_out[2^k - 1] receives them level by level (popcount 1, 2, ..., k),
 * level_off_out[k + 2] the first index of every level (entry 0 is 0, entry k + 1 the total).
 * Within a level, neighbours differ by one node swapped for another (revolving-door order):
 * the sweep kernel that takes two node sets per warp relies on it. */
pp_status pp_debug_mask_order(int32_t k, uint32_t *masks_out, uint32_t *level_off_out);

/* Measurement hook: issue rate of the packed 16-bit min/max instructions the sweep consists of, on
 * the current device.  One block of 1024 threads per SM runs `iters` trips of 64 dependent-chain
 * instructions per thread on registers only, timed with the SM's own cycle counter; the median over
 * the SMs gives *warp_instr_per_clk_per_sm (host).  op: 0 = two-input packed minimum and maximum in
 * turn, 1 = three-input packed minimum, 2 = three-input packed maximum.  The ALU bound of the search's roofline is this
 * rate x 32 lanes x 2 elements x SMs x clock.  Synchronous, legacy default stream; allocates and
 * frees a few hundred bytes of device memory. */
pp_status pp_debug_minmax_rate(int32_t op, int32_t iters, double *warp_instr_per_clk_per_sm);

/* Test hook: make the nth device allocation the library attempts from now on (1 = the next one)
 * report "out of memory" without asking the driver; 0 clears a pending request.  Lets a test see
 * PP_ERR_NOMEM come back from pp_problem_create, pp_solve_exact and the host-pointer entry points on
 * a device that has memory to spare. */
pp_status pp_debug_fail_alloc(int32_t nth);

/* Force (1) or forbid (0) the generic sweep kernel; 2 = automatic choice among the kernels that
 * take one source mask per warp (the two-mask kernel is left out); 3 = the two-mask kernel on every
 * level it can run, however small; -1 restores the automatic choice.  Meant for tests that want
 * every kernel checked on the same instance. */
pp_status pp_problem_force_generic(pp_problem *p, int32_t mode);

/*
 * Exact search that allocates nothing (the paper has no counterpart; this entry point exists
 * for the library's users, not for the method).
 *
 * Who needs it: code that must not, or cannot, call cudaMalloc at this point -- a process
 * whose whole device heap was handed to a framework's caching allocator at start-up, or a
 * plug-in that is only allowed to launch work.  pp_problem_create / pp_solve_exact allocate
 * device and pinned memory; this call does not.  It performs the same search with the same
 * kernels (the generic sweep) and gives bit-identical results, but every byte of device
 * scratch (inputs copy, gamma and rank tables, state table) comes from one array of
 * PP_STATIC_SCRATCH_BYTES that is compiled into the library.  Every GPU that loads the library
 * holds that array until the process exits, whether or not this call is ever made.
 *
 *   layer_out_bits, layer_mem_bytes  host [L];  node_mem_bytes host [k];  bw_kbps host [k*k]
 *   solution_dev   device, sizeof(pp_solution), 8-byte aligned: receives the result record
 *   cuda_stream    a cudaStream_t (NULL = legacy default stream).  The inputs, and a few small
 *                  tables this call prepares on its own stack, are pageable host memory: each
 *                  cudaMemcpyAsync of them is a staged copy that blocks the host until the
 *                  bytes have left the host buffer (the buffers may be reused as soon as the
 *                  call returns).  The kernels are then queued on the stream and the call
 *                  returns without waiting for them.
 * Limits: k <= 14, L <= PP_MAX_L, and the scratch the instance needs (dominated by the state
 * table, k * 2^k rows of L elements of 2 or 4 bytes) must fit PP_STATIC_SCRATCH_BYTES; anything
 * larger returns PP_ERR_LIMIT before any work is queued (k = 10, L = 50 needs about 1.1 MB;
 * k = 14, L = 100 about 52 MB).  Host-side preparation uses about 100 KB of stack.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress,
 * with that device current) and caches it; that first call should come before any stream
 * capture.  Nothing in this call was written for, or tried under, stream capture: the host-side
 * staging above and the per-launch attribute calls are ordinary eager-mode work.
 * All calls share the one array and it keeps the previous call's contents; the library resets
 * the words that must start clean itself.  Two calls whose GPU work overlaps (different
 * streams, or different host threads) race on the array: serialise them.
 * No cudaMalloc, cudaFree, cudaMallocHost or other allocating routine is called.
 */
#define PP_STATIC_SCRATCH_BYTES (64u << 20)
pp_status pp_solve_exact_static(int32_t L, const uint64_t *layer_out_bits,
                                const uint64_t *layer_mem_bytes, int32_t k,
                                const uint64_t *node_mem_bytes, const uint32_t *bw_kbps,
                                pp_solution *solution_dev, void *cuda_stream);

const char *pp_status_str(pp_status s);

#ifdef __cplusplus
}
#endif
#endif /* PP_H */
