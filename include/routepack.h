/*
 * routepack.h -- C ABI of the B200 (sm_100a) RoutePack planner hot path.
 *
 * The library plans one optimizer-step window at a time on one GPU: it reduces the
 * routing-replay counts to per-layer expert loads, places experts on EP ranks with the
 * layer-local LPT rule, projects every sample's demand onto physical ranks, picks the
 * row count and a length-only seed layout, scores layouts with the EDP-shard-aware
 * objective and refines a population of layouts by population annealing.  Every step
 * runs in CUDA kernels of this library; there is no CPU fallback.
 *
 * Conventions
 *  - All functions return RP_OK (0) or a negative rp_status; none throws, prints, aborts
 *    or traps.  rp_strerror() names a status.  Calling out of order gives RP_ERR_STATE.
 *  - Array arguments are plain pointers to HOST or DEVICE memory (either is accepted for
 *    every array, resolved with the CUDA unified-addressing rules).  The caller owns every
 *    buffer it passes.  Output arrays are complete when the call returns (each call
 *    synchronises its stream before returning).
 *  - Scalars and structs are passed from host memory.
 *  - A context belongs to the device that was current in rp_window_load and to the
 *    stream given there; calls on one context must not overlap.
 *  - Layouts are int32 arrays cell_of[N] with cell = row * dp_width + dp_slot.
 *  - Scores are int64 triples in fixed point: (max_g U_g, sum_g U_g, max_{r,g} J_{r,g})
 *    multiplied by 2^8 * token_cap^2, and the same triple as doubles divided by that scale.
 */
#ifndef ROUTEPACK_H_
#define ROUTEPACK_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RP_OK = 0,
    RP_ERR_ARG = -1,           /* NULL or out-of-range scalar argument                    */
    RP_ERR_SHAPE = -2,         /* E not a multiple of P, N < D, bad EDP partition, ...     */
    RP_ERR_CONSERVATION = -3,  /* some t_i outside [1,C], negative count, or sum_e a != k*t */
    RP_ERR_INFEASIBLE = -4,    /* no row count R <= N/D admits the length-only packing      */
    RP_ERR_RANGE = -5,         /* fixed-point range or on-chip memory budget exceeded       */
    RP_ERR_CUDA = -6,          /* a CUDA call failed; see rp_last_cuda_error()              */
    RP_ERR_STATE = -7,         /* call out of order                                         */
    RP_ERR_TIMEOUT = -8,       /* rp_anneal: a bounded device-side wait ran out (see there) */
    RP_ERR_INVALID_PLAN = -9   /* rp_best: the incumbent failed validation                  */
} rp_status;

typedef struct rp_ctx rp_ctx;  /* opaque; owns all device state of one window */

#define RP_MAX_STAGES 8

/* Problem statement (Sections 3.1-3.4 of the paper). */
typedef struct {
    int32_t n_samples;          /* N                                                        */
    int32_t n_layers;           /* L  MoE layers                                            */
    int32_t n_experts;          /* E  logical experts per layer                             */
    int32_t top_k;              /* k  assignments per token per layer                       */
    int32_t token_cap;          /* C  tokens per cell                                       */
    int32_t dp_width;           /* D  controller DP slots per execution row                 */
    int32_t ep_width;           /* P  physical EP ranks; E % P == 0                         */
    const int32_t *edp_of_dp;   /* HOST [D]: DP slot -> EDP shard g in [0,G), every g used;
                                   NULL = identity (G = D)                                  */
    int32_t n_stages;           /* attention stage types, 1..RP_MAX_STAGES                  */
    const double *alpha;        /* HOST [n_stages] token-linear coefficients  (>= 0)        */
    const double *beta;         /* HOST [n_stages] token-pair coefficients    (>= 0)        */
    int32_t pop_size;           /* P_pop population members                                 */
    int32_t min_rows;           /* optional lower bound on the row count; 0 = none          */
    uint64_t seed;              /* Philox key of the annealing random streams               */
} rp_config;

/* Search budget (Section 4.1.2, Algorithm 3). T_n = t0 * t_ratio^n. */
typedef struct {
    int32_t n_levels;           /* temperature levels N                                     */
    int32_t steps_per_level;    /* proposals K per chain per level                          */
    double t0;                  /* first temperature, in relative-energy units              */
    double t_ratio;             /* geometric ratio in (0,1]                                 */
    double p_reloc;             /* relocation probability rho in [0,1]                      */
    double p_guide;             /* guided-proposal probability in [0,1] (paper: 0.8)        */
} rp_anneal_params;

typedef struct {
    int64_t proposed, feasible, accepted, improved;  /* summed over chains and levels       */
    double ms_chains;           /* device time of all levels (chain kernels incl. the level
                                   barrier that runs in their last CTA, and launch gaps)    */
    int64_t move_bytes;         /* algorithmic bytes of the feasible moves: rank-load slices
                                   and demand rows read, slices written on accept           */
    int64_t gather_bytes;       /* rank-load bytes read+written for members that resampling
                                   replaced by another member's state                       */
    int64_t staging_bytes;      /* rank-load bytes moved between global and shared memory for
                                   members that kept their own state (windows whose rank loads
                                   live on chip during a level); 0 otherwise                 */
    int64_t kernel_launches;    /* kernels this call launched                                */
} rp_anneal_stats;

/* Routing-replay input (Eq. routing-replay-input): creates a context, copies host arrays
 * to the device (device arrays are adopted without a copy and must stay valid until
 * rp_pack_rows returns: rp_place_experts may leave its work queued on the stream) and checks 1 <= t_i <= C, a >= 0 and sum_e a[i][l][e] == k*t_i.
 *   lengths [N] int32; demand [N][L][E] int32, expert index fastest.
 *   cuda_stream: a cudaStream_t (NULL = default stream).
 * The placement, projection and packing kernels depend on nothing but these inputs and are queued
 * on the stream right behind the checks, so the GPU is already working on them while the host
 * waits for the verdict (packing, which reads only the lengths, on an internal side stream that
 * forks from and joins the context's stream inside this call); rp_place_experts and
 * rp_pack_rows then hand their results over (and compute them themselves when called again).
 * On failure *out is NULL. */
int rp_window_load(rp_ctx **out, const rp_config *cfg, const int32_t *lengths,
                   const int32_t *demand, void *cuda_stream);

/* Layer-wise expert placement (Section 3.3, Algorithm 1) and demand projection
 * (Eq. physical-rank-demand).  Aggregates L[l][e] = sum_i a[i][l][e], places each layer's
 * experts by decreasing load on the least-loaded rank with a free slot (ties: lower expert
 * id, lower rank id; exactly E/P experts per rank; slot = rank*(E/P) + arrival index), then
 * computes q[i][l][p].
 *   pi [L][E] int32 out, nullable: physical slot of logical expert e.
 *   rank_load [L][P] int64 out, nullable: aggregate load G[l][p] under pi.
 * Outputs (host or device memory) are complete on return; with both NULL the call only queues
 * its work on the context's stream. */
int rp_place_experts(rp_ctx *ctx, int32_t *pi, int64_t *rank_load);

/* Row count and seed population (Section 3.2; Algorithm 2, first line and last loop).
 * R_lb = max(1, min_rows, ceil(sum t / (C*D))); for R = R_lb, R_lb+1, ... first-fit-decreasing
 * into R*D cells (the R*D longest samples open the cells, each later sample goes to the
 * lowest-numbered cell it fits); the first R that packs is R*.  certified = 1 iff R* == R_lb
 * (then it is the minimum).  Every population member starts as this layout.
 *   n_rows, certified: HOST scalars out (nullable). */
int rp_pack_rows(rp_ctx *ctx, int32_t *n_rows, int32_t *certified);

/* Randomized fixed-row seeds (Algorithm 2, the trial loop; the pairing and canonical-selection
 * operators are not applied).  Optional, between rp_pack_rows and rp_anneal.  Member 0 keeps the
 * length-only seed; member j >= 1 runs trial j: WindowShuffle (emit a uniformly chosen one of the
 * next choice_width samples in decreasing-length order) feeds RandomizedBestFit (the first R*D
 * emitted samples open the cells; each later one takes a uniformly chosen one of the leading
 * choice_width cells it fits in, ranked fuller first, then fewer samples, then lower index);
 * a trial with no feasible cell is dropped and its member keeps the length-only seed.  All
 * members are scored from scratch; the incumbent becomes the best member (lowest index on ties).
 *   choice_width in [1, 32]; n_own: HOST out, members that carry their own trial (nullable). */
int rp_seed_population(rp_ctx *ctx, int32_t choice_width, int32_t *n_own);

/* EDPAwarePair on the current population (Section 4.1.1; Algorithm 2, third construction
 * operator).  Optional, between rp_pack_rows and rp_anneal (after rp_seed_population when both are
 * used).  Member 0 is left as it is; in every member j >= 1 each completed cell keeps its samples
 * and moves to a new (row, DP slot):
 *   - profile w_b[l][p] = sum of q[i][l][p] over the cell's samples; cells are taken by decreasing
 *     routed-token peak max w_b (ties: lower cell index);
 *   - every empty slot gets the insertion key (increase of sum_l max_p of its row-shard's rank
 *     load, largest such peak afterwards); slots are ranked by ascending key, ties by lower index;
 *   - rank-decaying sampling among the leading min(choice_width, #empty) slots: rank 0 with
 *     probability 1/2, rank 1 with 1/4, ..., the remainder on the last rank (the paper names the
 *     rule without giving its law; this is one reading of it).  Draw: Philox(h, 0, j, 6) for the
 *     h-th cell placed.
 * All members are scored from scratch; the incumbent becomes the best member (lowest index on ties).
 *   choice_width in [1, 32]; n_changed: HOST out, members whose layout changed (nullable).
 * RP_ERR_STATE outside stage 3, RP_ERR_RANGE when the per-member tables exceed shared memory. */
int rp_pair_population(rp_ctx *ctx, int32_t choice_width, int32_t *n_changed);

/* Canonicalize + CanonicalMap + QualityDiversitySelect with the current population as the
 * candidate set (Section 4.1.1; Algorithm 2, last lines).  Optional, between rp_pack_rows and
 * rp_anneal, after the seeding calls above.
 *   - signature: a cell is named by its smallest sample; inside a row the cells of one EDP shard
 *     are listed by name over the shard's slots, rows are listed by their smallest sample.  Members
 *     with equal signatures are the same plan up to row order and exchangeable DP slots; the class
 *     is represented by its lowest score, then lowest index.
 *   - the selection starts from the representative with the lowest score and then repeatedly takes
 *     the one that maximises  (distance to the nearest selected) - ((eta_q16 * gap) >> 16),
 *     gap = floor((S0 - S0_best) * 2^20 / S0_best), ties by lower index.
 *   - distance (Q20 units): cell co-assignment + row co-assignment (1 - pairs together in both /
 *     pairs together in either) + a Sliced-Wasserstein sketch: L1 distance of the sorted projections
 *     of the Q16 row features (tokens/(C*D), squared lengths/(C*C*D), busiest rank of every (shard,
 *     layer)/(k*C*slots of the shard)) onto n_proj +-1 vectors (sign f of vector k = top bit of
 *     Philox(f, 0, k, 7)), times 16 / (n_proj * R * F).
 *   - new member m = the (m mod n_distinct)-th selected representative.
 * The paper names the ingredients of the distance, eta, the feature matrix and the projections
 * without fixing them: the mixing (equal weights), the features and the sign vectors are this
 * library's reading.  Cost grows with the square of the number of distinct members.
 *   n_proj in [1, 64]; eta_q16 >= 0; n_distinct HOST out (nullable); order HOST out [P_pop],
 *   former member index of every new member (nullable). */
int rp_select_population(rp_ctx *ctx, int32_t n_proj, int64_t eta_q16, int32_t *n_distinct, int32_t *order);

/* Algorithm 2 as one operation (Section 4.1.1, all lines): M = n_candidates fixed-row candidates,
 *   candidate 0 = x_length (the length-only seed),
 *   candidate 1 = x_paired = the lower-scoring of x_length and EDPAwarePair(x_length) (x_length on ties),
 *   candidate t >= 2 = EDPAwarePair(trial t), trial t = WindowShuffle -> RandomizedBestFit with the
 *     random streams of member t of rp_seed_population / rp_pair_population (a trial with no feasible
 *     cell falls back to the length-only seed before it is paired),
 * then CanonicalMap over all M and QualityDiversitySelect as in rp_select_population; population
 * member m becomes the (m mod n_distinct)-th selected plan.  Between rp_pack_rows and rp_anneal;
 * replaces whatever the population held.  The incumbent becomes the best member.
 *   n_candidates in [2, 65536] (may be smaller or larger than the population); choice_width in
 *   [1, 32]; n_proj in [1, 64]; eta_q16 >= 0.  n_distinct: HOST out (nullable); picked: HOST out
 *   [P_pop], candidate index of every member (nullable).
 * Cost grows with the square of the number of distinct candidates (see rp_select_population). */
int rp_init_population(rp_ctx *ctx, int32_t n_candidates, int32_t choice_width, int32_t n_proj, int64_t eta_q16,
                       int32_t *n_distinct, int32_t *picked);

/* Full evaluation of layouts (Section 3.4-3.5: Eqs. cell-token-statistics,
 * stage-aware-attention, row-expert-load, row-expert-cost, lexicographic-score).
 *   layouts [n][N] int32 cell ids, or NULL to score the current population (n = pop_size).
 *   score_fx [n][3] int64 out, nullable; score_f64 [n][3] double out, nullable.
 * Layouts with a cell id outside [0, R*D) give RP_ERR_ARG. */
int rp_eval_population(rp_ctx *ctx, const int32_t *layouts, int32_t n, int64_t *score_fx,
                       double *score_f64);

/* The same scores as rp_eval_population, for callers that must not allocate device memory
 * once they are running: a planner called from inside a training or serving loop whose
 * framework has already handed all free device memory to its own pool, or from a section
 * where an allocation would stall the whole device (cudaMalloc and cudaFree synchronise it).
 * The paper has no counterpart; this is a deployment variant of the full evaluation.
 * It calls no cudaMalloc/cudaFree or any allocating routine: its working memory (16-bit cell
 * ids, row-shard sums, arrival counters; about 1.3 MiB) is a fixed array inside the library
 * image, present on every GPU that loads the library until the process exits.
 *   layouts [n][N] int32, score_fx [n][3] int64 (nullable), score_f64 [n][3] double
 *   (nullable): all three must be DEVICE pointers (a host array would need a staging buffer).
 *   Limits: n <= 1024, n*N <= 524288, n*R*G <= 32768; beyond them the call returns
 *   RP_ERR_RANGE and does nothing (use rp_eval_population).
 * The first call on a device looks up the device address of the fixed array
 * (cudaGetSymbolAddress); make that first call before any stream capture.  The context's
 * device must be the current device (RP_ERR_STATE otherwise).  All calls in the process share
 * the one array and it keeps the previous call's contents (the call clears the part that must
 * start at zero): two calls whose kernels overlap on the GPU, from different contexts or
 * streams, race on it, so issue them one after the other. */
int rp_eval_layouts_noalloc(rp_ctx *ctx, const int32_t *layouts, int32_t n, int64_t *score_fx,
                            double *score_f64);

/* Fixed-row population annealing (Algorithm 3): n_levels temperature levels; at each level
 * every member runs steps_per_level guided swap/relocation proposals with incremental
 * rescoring and the Metropolis rule, the incumbent takes any strictly better
 * trajectory-best plan, and (except after the last level) the population is resampled
 * systematically with Boltzmann weights.  May be called again to continue from the
 * current population; level indices of the random streams restart at 0 on each call.
 * Before it returns the call also validates and fully rescores its incumbent (the checks of
 * rp_best) in the same stream, so that a following rp_best has nothing left to compute.
 *   stats: HOST out, nullable.
 * Every wait of a chain on its asynchronous copies is bounded.  If one runs out, that chain stores
 * nothing, the level's barrier and all later levels are skipped, and the call returns
 * RP_ERR_TIMEOUT with the device and the context intact but the population undefined: call
 * rp_pack_rows again to start over from the seed, or rp_destroy. */
int rp_anneal(rp_ctx *ctx, const rp_anneal_params *params, rp_anneal_stats *stats);

/* Validate(x*) and the non-regression assertion that close Algorithm 3 (Section 4.1.3: the
 * returned plan is the archived incumbent, checked before it is handed to the trainer): coverage,
 * capacity, non-empty cells, cached score equals a full rescoring, not worse than the best seed;
 * then return it.
 *   cell_of_sample [N] int32 out, nullable; score_fx [3], score_f64 [3] out, nullable.
 * RP_ERR_INVALID_PLAN when a check fails.  Outputs are complete on return.  Right after
 * rp_anneal the checks are already done and the call only hands the results over. */
int rp_best(rp_ctx *ctx, int32_t *cell_of_sample, int64_t *score_fx, double *score_f64);

/* Load-balance diagnostics of the paper's evaluation section for one layout (Eq. global-ep-cv,
 * the EP peak sum and tail peak, Eq. ep-efficiency, and the attention / joint proxies of its
 * mechanism table).  W is the rank-load tensor of the layout under the committed placement.
 *   cv_identity / cv_placed: mean over layers of std_p(G[l][p]) / mean_p(G[l][p]) of the
 *     aggregate rank loads, with expert e on rank e/(E/P), and under the LPT placement;
 *   s_ep = sum_{r,l} max_{g,p} W;  t_ep = max W;  n_ep = sum_{r,l} max_g sum_p W;
 *   eta_ep = n_ep / (P * s_ep);  attention = sum_{r,g} A_{r,g};  joint = max_g sum_r J_{r,g}.
 *   layout [N] int32 (host or device), NULL = the incumbent.  out: HOST struct. */
typedef struct {
    double cv_identity, cv_placed;
    int64_t s_ep, t_ep, n_ep;
    double eta_ep, attention, joint;
} rp_diag;
int rp_diagnostics(rp_ctx *ctx, const int32_t *layout, rp_diag *out);

/* Frees the context.  Its device memory goes back to a per-device cache inside the library
 * (so that the next window does not pay for allocation); rp_release_cached_memory() returns
 * that cache to the driver. */
void rp_destroy(rp_ctx *ctx);
int rp_release_cached_memory(void);
const char *rp_strerror(int status);
/* cudaError_t value of the last failed CUDA call on this thread (0 if none). */
int rp_last_cuda_error(void);

/* ---- inspection hooks (the paper has no counterpart; used by the parity tests) -------- */
typedef enum {
    RP_DUMP_LAGG = 1,        /* int64 [L][E]                                               */
    RP_DUMP_Q = 2,           /* int32 [N][L][P]                                            */
    RP_DUMP_SEED_LAYOUT = 3, /* int32 [N]                                                  */
    RP_DUMP_POPULATION = 4,  /* int32 [P_pop][N]  current layouts                          */
    RP_DUMP_W = 5,           /* int32 [R][G][L][P] of population member `index`            */
    RP_DUMP_CELL_T = 6,      /* int64 [R*D] token sums of member `index` (recomputed)      */
    RP_DUMP_CELL_Q = 7,      /* int64 [R*D] squared-length sums of member `index`          */
    RP_DUMP_CELL_CNT = 8,    /* int32 [R*D]                                                */
    RP_DUMP_ESUM = 9,        /* int64 [R][G]  sum_l max_p W of member `index`              */
    RP_DUMP_TRACE_TERM = 10, /* int64 [n_levels][P_pop][3] terminal scores, last rp_anneal */
    RP_DUMP_TRACE_BEST = 11, /* int64 [n_levels][P_pop][3] trajectory-best scores          */
    RP_DUMP_TRACE_BEST_STEP = 12, /* int32 [n_levels][P_pop], 0 = level start              */
    RP_DUMP_TRACE_DIGEST = 13,    /* uint64 [n_levels][P_pop] digest of accepted moves     */
    RP_DUMP_TRACE_ANC = 14,       /* int32 [n_levels-1][P_pop] resampling ancestors        */
    RP_DUMP_TRACE_INCUMBENT = 15, /* int64 [n_levels][3]                                   */
    RP_DUMP_SELECT_DIST = 17, /* int64 [P_pop][P_pop] plan distances between the representatives
                                 of the last rp_select_population (0 elsewhere); inspection hook on */
    RP_DUMP_EVAL_W = 16      /* int32 [R][G][L][P] of layout `index` of the last
                                rp_eval_population call with explicit layouts (n <= 64)    */
} rp_dump_what;
/* Knobs that steer the annealing kernels onto paths that full-size windows or failures reach,
 * so that small tests can cover them; all 0 (off) by default.
 *   RP_KNOB_BARRIER_WORKSPACE: shared-memory bytes (multiple of 16, >= 64) the level barrier may
 *     use; a small value sends its cumulative weights, cell bookkeeping and incumbent replay
 *     through their global-memory forms.
 *   RP_KNOB_WAIT_POLLS: polls after which a chain's wait on its asynchronous copies gives up
 *     (default 2^22); a chain's wait for the other chains of a launch that runs all levels then
 *     gives up after that many microseconds (default 2 s + 50 us per step of a level).
 *   RP_KNOB_STALL_ONE_CHAIN: chain 0 waits once more, after its copies have landed, on a barrier
 *     phase that nothing completes: the wait runs out and rp_anneal returns RP_ERR_TIMEOUT.
 *   RP_KNOB_LAUNCH_PER_LEVEL: how rp_anneal launches windows whose chains can all be resident at
 *     once (rank loads on chip, at most 256 members).  0 or 2 = one launch for all levels (lowest
 *     latency of a single plan); 1 = one launch per level (two windows planned at once on two
 *     streams then share the GPU, which two launches of the first kind cannot).
 *   RP_KNOB_RANK_LOAD_SLICES (set before rp_pack_rows): how windows with L*P > 512 keep the rank
 *     loads of the population.  0 or 1 = shared slices with copy-on-write (the default), 2 = one
 *     private cell per member, copied whole when resampling replaces the member.
 *   RP_KNOB_CHAIN_KERNEL: which chain kernel windows use whose rank loads live in the slice pool
 *     (not on chip).  0 = one warp per chain, except for windows with L*P <= 512 and at most 592
 *     members, which finish sooner with several warps per chain; 1 = always several warps per
 *     chain; 2 = always one warp per chain. */
typedef enum { RP_KNOB_BARRIER_WORKSPACE = 1, RP_KNOB_WAIT_POLLS = 2, RP_KNOB_STALL_ONE_CHAIN = 3,
               RP_KNOB_RANK_LOAD_SLICES = 4, RP_KNOB_LAUNCH_PER_LEVEL = 5, RP_KNOB_CHAIN_KERNEL = 6 } rp_knob;
int rp_debug_set_knob(rp_ctx *ctx, int knob, int64_t value);
/* Device time of the stages that have no statistics struct of their own.  After
 * rp_debug_set_stage_timing(1) (process-wide; contexts loaded later record CUDA events around the
 * kernels, a few microseconds of host time per call), rp_debug_stage_times synchronises the
 * context's stream and fills ms[6], milliseconds, -1 where the stage has not run on this context:
 *   [0] input checks + aggregate demand (K1)   [1] placement, Algorithm 1 (K2)   [2] projection (K3)
 *   [3] row count + length-only seed (runs beside [0]-[2] on a side stream)
 *   [4] seed evaluation and tables in rp_pack_rows   [5] validation + rescoring of the incumbent. */
int rp_debug_set_stage_timing(int on);
int rp_debug_stage_times(rp_ctx *ctx, double *ms);
/* Per-level traces (RP_DUMP_TRACE_*) are recorded by rp_anneal calls made after
 * rp_debug_set_trace(ctx, 1); off by default (the copies cost a few microseconds per level). */
int rp_debug_set_trace(rp_ctx *ctx, int on);
/* Copies the named array into buf (host or device); bytes must equal its size. */
int rp_debug_dump(rp_ctx *ctx, int what, int32_t index, void *buf, int64_t bytes);
/* Element-wise device evaluation of the integer functions used by the accept test and the
 * resampling weights: out[i] = -log2((x[i]+1)/2^32) in Q32, and out[i] = 2^(-z[i]) in Q32.
 * x, z, out: host or device arrays of n elements. */
int rp_debug_nl2(const uint32_t *x, uint64_t *out, int64_t n);
int rp_debug_exp2neg(const uint64_t *z, uint64_t *out, int64_t n);
/* out[i][0..3] = Philox4x32-10(counter ctr[i][0..3], key) on the device. */
int rp_debug_philox(const uint32_t *ctr, const uint32_t key[2], uint32_t *out, int64_t n);
/* Read bandwidth, in GB/s, of a zeroed buffer of `bytes` (1 MiB .. 2 GiB) that every thread of a
 * full grid sums `reps` times over with 16-byte loads: with a buffer that fits L2 this is the
 * measured L2 read rate that kernels whose operands L2 serves are set against.  Allocates and
 * frees its own buffer; runs on the default stream of the current device. */
int rp_debug_l2_read_rate(int64_t bytes, int32_t reps, double *gb_per_s);
/* Which chain kernel rp_anneal runs for this context (valid after rp_pack_rows; inspection only):
 * 0 = warp per candidate (k_anneal_wpc), 1 = 128 threads per chain (k_anneal_level), 2 = warp per
 * chain (k_anneal_warp). */
int rp_debug_chain_kernel(rp_ctx *ctx, int32_t *which);
/* Number of kernels this library has launched in this process so far. */
int64_t rp_debug_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ROUTEPACK_H_ */
