// Internal declarations of the RoutePack B200 library: context, launch wrappers and the
// device-side integer helpers (random numbers, -log2, 2^-z, score order, energy).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "routepack.h"

#define RP_FBITS 8              // fraction bits of the attention coefficients
#define RP_MAX_EDP 1024         // G upper bound
#define RP_MAX_EP 1024          // P upper bound

typedef unsigned long long u64;
typedef long long i64;
typedef unsigned int u32;

// ---------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------
extern thread_local int g_rp_last_cuda_error;
extern long long g_rp_launches;
#define RP_CUDA(call)                                                    \
    do {                                                                 \
        cudaError_t e_ = (call);                                         \
        if (e_ != cudaSuccess) {                                         \
            g_rp_last_cuda_error = (int)e_;                              \
            return RP_ERR_CUDA;                                          \
        }                                                                \
    } while (0)
#define RP_TRY(call)                                                     \
    do {                                                                 \
        int s_ = (call);                                                 \
        if (s_ != RP_OK) return s_;                                      \
    } while (0)

// ---------------------------------------------------------------------------------------
// problem constants handed to every kernel (fits in kernel-parameter space)
// ---------------------------------------------------------------------------------------
struct RpDims {
    int N, L, E, k, C, D, P, G, H, S;   // H = E / P experts per rank, S = attention stages
    int R, K, RG, LP;                   // rows, cells R*D, row-shards R*G, L*P (set after packing)
    int slices;                         // rank loads kept as shared slices (set after packing; see AnnealArgs)
    i64 ahat[RP_MAX_STAGES], bhat[RP_MAX_STAGES];
    i64 asum, bsum;                     // sums over stages (attention key of a cell)
    i64 SC;                             // 2^8 * C^2
    i64 EC;                             // 2^8 * C
};

// per-level schedule integers
struct RpLevel {
    u64 tau;        // floor(T_n * ln2 * 2^32)
    u64 cq;         // floor((1/T_{n+1} - 1/T_n) / ln2 * 2^16)
};

// Small state of one chain as one contiguous blob, laid out the same way in global and in
// shared memory so that a single bulk copy moves it.  Offsets in bytes from a 16-byte
// aligned base; `bytes` is a multiple of 16.
struct RpBlob {
    int off_Q;      // u64 [K]   squared-length sum per cell
    int off_Esum;   // i64 [RG]  sum_l max_p W
    int off_Afx;    // i64 [RG]  attention cost of the row-shard
    int off_Jfx;    // i64 [RG]  Afx + 2^8*C*Esum
    int off_U;      // i64 [G]   shard work
    int off_S;      // i64 [4]   score tuple and energy
    int off_T;      // int [K]   token sum per cell
    int off_cnt;    // int [K]   samples per cell
    int off_cell;   // u16 [N]   sample -> cell
    int off_wtab;   // int [RG]  slice of the rank-load pool that holds each row-shard (-1: windows whose rank loads
                    //           sit in one cell per member, see rp_uses_slices)
    int bytes;
};
// Tables that are the same for every chain of a plan (one block in global memory).
struct RpStatic {
    int off_dpl;    // int [D]   DP slots grouped by shard
    int off_dpo;    // int [G+1] start of each shard's group
    int off_t;      // int [N]   sample lengths (present when t_staged)
    int off_rg;     // u16 [K]   cell -> row-shard
    int off_g;      // u16 [K]   cell -> shard
    int off_row;    // u16 [K]   cell -> first cell of its row
    int bytes;
    int t_staged;
};

// one population buffer set (two of them: the level reads one and writes the other)
struct RpPopBuf {
    char *blob;                // [P_pop][blob.bytes]
};

// Events of the optional stage timing: begin/end of the check+reduce, placement, projection and
// packing kernels (rp_window_load), of the seed's evaluation and tables (rp_pack_rows) and of the
// validation + rescoring of the incumbent.
enum { RP_EV_K1_0, RP_EV_K1_1, RP_EV_K2_0, RP_EV_K2_1, RP_EV_K3_1, RP_EV_PACK_0, RP_EV_PACK_1, RP_EV_SEED_0, RP_EV_SEED_1,
       RP_EV_BEST_0, RP_EV_BEST_1, RP_STAGE_EVENTS };

struct rp_ctx {
    int device;
    cudaStream_t stream;
    int stage;                 // 1 loaded, 2 placed, 3 packed, 4 annealed at least once
    rp_config cfg;             // scalars only (pointers copied below)
    RpDims dm;
    int Ppop;
    // inputs
    const int *d_t;            // [N]
    const int *d_a;            // [N][L][E]
    int *own_t, *own_a;        // non-null when this context allocated the copies
    char *d_load_slab;         // one allocation behind the buffers sized by the window alone (freed by rp_destroy)
    char *d_pop_slab;          // one allocation behind the population buffers (sized after packing)
    int *d_edp;                // [D]
    int *d_dp_list;            // [D] DP slots grouped by shard
    int *d_dp_off;             // [G+1]
    // placement
    i64 *d_Lagg;               // [L][E]
    int *d_pi;                 // [L][E]
    int *d_inv;                // [L][E]  slot -> expert
    i64 *d_rank_load;          // [L][P]
    int *d_q;                  // [N][L][P]
    int *d_status;             // device status words (see RpStatusWord)
    // packing
    u64 *d_sort_keys;          // scratch for the length sort
    int *d_seed_layout;        // [N]
    int *d_order;              // [N] samples sorted by (-t, i)
    int *d_pack_out;           // [4]: R*, certified, R_lb, failure flag
    int Rstar, certified;
    i64 seed_score[3];
    // population
    RpPopBuf buf[2];
    int *d_W;                  // [2*P_pop][RG][LP] rank-load cells; a member's W sits in the cell wloc says
    int *d_wloc;               // [P_pop] cell of each member's current W (read through d_anc)
    int *d_wloc_next;          // [P_pop] cell each member works in during the next level
    int *d_le_scratch;         // [6*P_pop] ints for the level barrier's cell bookkeeping
    int *d_wref;               // [2*P_pop*RG] members that hold each slice when a level starts (slice mode)
    int *d_wcount;             // [2*P_pop*RG] the same while it is being counted; zero between two counts
    int *d_wfree;              // [2*P_pop*RG] slices nobody holds, handed out in this order during the level
    int *d_wfree_head;         // [2] next free-list entry to hand out, entries in the list
    RpBlob bl;
    RpStatic sl;
    char *d_static;            // static tables block
    int cur;                   // buffer holding the current population
    int *d_anc;                // [P_pop] which member of buf[cur] each slot continues from
    int *d_anc_next;           // [P_pop] written by the level barrier, swapped with d_anc
    int *d_done;               // arrival counter of the chain CTAs
    int *d_sync;               // arrival counter of the launch that runs all levels
    void *d_levels;            // per-level schedule integers on the device (RpLevelDev), levels_dev_cap of them
    int levels_dev_cap;
    // per-level results
    i64 *d_term;               // [P_pop][3]
    i64 *d_best;               // [P_pop][3]
    int *d_best_step;          // [P_pop]
    int *d_best_nlog;          // [P_pop]  accepted moves logged when the best was reached
    u64 *d_digest;             // [P_pop]
    uint2 *d_log;              // [P_pop][log_cap] accepted moves (sample, second | reloc<<31)
    int log_cap;
    u64 *d_F;                  // [P_pop] cumulative weights
    i64 *d_counters;           // [4]
    // incumbent
    int *d_inc_layout;         // [N]
    unsigned short *d_cand_layout;   // [P_pop][N] trajectory-best snapshots of the chains (warp-per-candidate kernel)
    int *d_inc_slot;           // [1]
    i64 *d_sel_dist;           // [P_pop][P_pop] plan distances of the last rp_select_population (inspection hook on)
    i64 *d_inc_score;          // [3]
    i64 *d_best_score;         // [3] full rescoring of the incumbent (validation)
    double *d_best_f64;        // [3] the same as the real-valued objective
    void *side;                // side stream + two events borrowed for the call that packs beside the placement (see RpSide)
    int eager_place, eager_pack;   // rp_window_load already queued the placement / packing kernels behind its checks
    int pack_out[4];           // R*, certified, R_lb, failure flag as read back with the load's verdict
    int best_ready;            // the incumbent has been validated and rescored since it last changed
    int best_verdict;          // RP_OK or RP_ERR_INVALID_PLAN of that validation
    // trace of the last rp_anneal call
    int trace_levels;
    int trace_on;              // keep per-level traces (inspection hook; off by default)
    int knob_level_launches;   // 1 = one launch per level even where one launch for all levels is possible
    int knob_chain_kernel;     // 1 = 128 threads per chain, 2 = one warp per chain, wherever the window allows both
    int knob_slices;           // inspection hook: 0 = automatic, 1 = slices wherever L*P > 512, 2 = never
    int knob_le_ws_cap, knob_wait_polls, knob_stall;   // inspection hooks (rp_debug_set_knob); 0 = off
    cudaEvent_t ev_stage[RP_STAGE_EVENTS];             // stage timing (rp_debug_set_stage_timing); null when off
    unsigned ev_recorded;                              // bit x: ev_stage[x] has been recorded
    i64 *d_tr_term, *d_tr_best, *d_tr_inc;
    int *d_tr_best_step, *d_tr_anc;
    u64 *d_tr_digest;
    // eval scratch
    i64 *d_eval_score;         // [n][3]
    double *d_eval_f64;        // [n][3]
    int *d_eval_W;             // W of explicitly evaluated layouts (n <= 64), for inspection
    int eval_W_n;
    unsigned short *d_eval_cells;
    i64 *d_eval_Esum;          // [n][RG] row-shard sums handed to the finishing CTA
    int *d_eval_tickets;       // [n] arrival counters, zero between launches
    size_t eval_cap;
    RpLevel *h_levels;         // host copy of the per-level schedule integers
    int levels_cap;
    i64 *h_pin;                // small pinned staging block for device->host scalars (64 x 8 bytes)
    i64 *d_seed_score;         // [3] best score of the initial population
};

enum RpStatusWord { RP_SW_BAD_SAMPLE = 0, RP_SW_BAD_LAYOUT = 1, RP_SW_VALIDATE = 2, RP_SW_TIMEOUT = 3, RP_SW_POOL = 4, RP_SW_COUNT = 8 };

// ---------------------------------------------------------------------------------------
// launch wrappers (each returns an rp_status; none synchronises)
// ---------------------------------------------------------------------------------------
int rp_launch_check_reduce(rp_ctx *c);
int rp_launch_lpt(rp_ctx *c);
int rp_launch_project(rp_ctx *c);
int rp_launch_pack(rp_ctx *c, int Rlb_hint);
int rp_launch_eval(rp_ctx *c, const unsigned short *cells, int n, int *W_out, char *blob_out,
                   i64 *score_out, double *f64_out);
int rp_launch_build_static(rp_ctx *c);
int rp_launch_seed_trials(rp_ctx *c, int width, int *layouts, int *ok);
int rp_launch_edp_pair(rp_ctx *c, const int *lay_in, int *lay_out, int *prof, int first, int count, int width);
int rp_launch_pack_on(rp_ctx *c, cudaStream_t stream);
int rp_launch_pick_best(rp_ctx *c, const i64 *scores, const int *layouts, int n, i64 *best_score_out);
int rp_get_pool(int device, cudaMemPool_t *out);     // the library's stream-ordered pool of a device
void rp_make_layouts(const RpDims &dm, RpBlob *bl, RpStatic *sl);
bool rp_uses_slices(const RpDims &dm);
int rp_slice_mode(const RpDims &dm, int knob);
void rp_decide_layouts(rp_ctx *c);
int rp_launch_slice_gc(rp_ctx *c);
int rp_launch_cells_from_layouts(rp_ctx *c, const int *layouts, int n, unsigned short *cells);
// Stream-ordered device memory from the device's pool (n elements of T; freed on the context's stream).
template <class T>
static inline int dev_alloc(rp_ctx *c, T **p, size_t n)
{
    *p = nullptr;
    if (n == 0) n = 1;
    cudaMemPool_t pool;
    RP_TRY(rp_get_pool(c->device, &pool));
    RP_CUDA(cudaMallocFromPoolAsync((void **)p, n * sizeof(T), pool, c->stream));
    return RP_OK;
}
static inline void dev_free(rp_ctx *c, void *p) { if (p) cudaFreeAsync(p, c->stream); }

// Carves 256-byte aligned pieces out of one allocation: first pass (base == nullptr) adds up the
// sizes, second pass hands out the pointers.
struct RpSlab {
    char *base;
    size_t off;
    template <class T>
    void take(T **p, size_t n)
    {
        if (n == 0) n = 1;
        if (base) *p = (T *)(base + off);
        off = (off + n * sizeof(T) + 255) & ~(size_t)255;
    }
};

int rp_launch_select(rp_ctx *c, int *lay, int *out, const i64 *score, int n_proj, i64 eta_q16, int *order,
                     int *n_distinct, i64 *dist);
bool rp_uses_wpc(const RpDims &dm);
bool rp_uses_warp_chains(const rp_ctx *c);
int rp_launch_anneal_level(rp_ctx *c, int level, int n_levels, const rp_anneal_params *prm, u64 rho_q32, u64 guide_q32);
int rp_launch_anneal_all(rp_ctx *c, int n_levels, const rp_anneal_params *prm, u64 rho_q32, u64 guide_q32, int *done);
int rp_upload_levels(rp_ctx *c, int n_levels);
int rp_launch_validate(rp_ctx *c);
int rp_anneal_smem_bytes(const rp_ctx *c, int *threads, size_t *bytes);

// ---------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__

// Philox4x32-10 (Salmon et al., SC'11): counter (c0..c3), key (k0,k1) -> 4 words.
__device__ __forceinline__ uint4 rp_philox(u32 c0, u32 c1, u32 c2, u32 c3, u32 k0, u32 k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        u32 hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        u32 hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        u32 n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// floor(x * n / 2^32): uniform index in [0, n)
__device__ __forceinline__ int rp_pick(u32 x, int n) { return (int)__umulhi(x, (u32)n); }

// -log2((x+1)/2^32) in unsigned Q32; 24 fraction bits by square-and-compare, truncated.
__device__ __forceinline__ u64 rp_nl2(u32 x)
{
    u64 v = (u64)x + 1ull;
    int e = 63 - __clzll((i64)v);
    u64 m = v << (63 - e);
    u32 frac = 0;
#pragma unroll 1
    for (int i = 0; i < 24; ++i) {
        u64 sq = __umul64hi(m, m);
        u32 bit = (u32)(sq >> 63);
        frac = (frac << 1) | bit;
        m = bit ? sq : (sq << 1);
    }
    return ((u64)(32 - e) << 32) - ((u64)frac << 8);
}

// floor(2^63 * 2^(-2^-i)), i = 1..24  (csrc/gen_exp2_consts.py)
__device__ __constant__ const u64 RP_EXP2_Q63[24] = {
    0x5A827999FCEF3242ULL, 0x6BA27E656B4EB57AULL, 0x75606373EE921C97ULL,
    0x7A92BE8A92436616ULL, 0x7D41D96DB915019DULL, 0x7E9F06067A4360BAULL,
    0x7F4F08AE3DC7C425ULL, 0x7FA765ACA88F6452ULL, 0x7FD3AB290E46D768ULL,
    0x7FE9D3A8E07BF085ULL, 0x7FF4E9597BED93AAULL, 0x7FFA748DFF8DC61EULL,
    0x7FFD3A3F50020332ULL, 0x7FFE9D1DBC0A75A9ULL, 0x7FFF4E8E6306ED58ULL,
    0x7FFFA74712C3CDFDULL, 0x7FFFD3A381B1FA28ULL, 0x7FFFE9D1BEED0189ULL,
    0x7FFFF4E8DEFB81D7ULL, 0x7FFFFA746F5F012FULL, 0x7FFFFD3A37A7D0A8ULL,
    0x7FFFFE9D1BD1FC58ULL, 0x7FFFFF4E8DE8832DULL, 0x7FFFFFA746F422D6ULL,
};

// 2^(-z), z unsigned Q32 -> Q32 (2^32 = 1.0); 24 fraction bits of z are used.
__device__ __forceinline__ u64 rp_exp2neg(u64 z)
{
    u64 ip = z >> 32;
    if (ip >= 32) return 0;
    u64 acc = 1ull << 63;
#pragma unroll 1
    for (int i = 1; i <= 24; ++i) {
        if ((z >> (32 - i)) & 1ull) {
            u64 c = RP_EXP2_Q63[i - 1];
            // (acc * c) >> 63 with a 128-bit product
            acc = (__umul64hi(acc, c) << 1) | ((acc * c) >> 63);
        }
    }
    return (acc >> 31) >> ip;
}

__device__ __forceinline__ bool rp_lex_less(i64 a0, i64 a1, i64 a2, i64 b0, i64 b1, i64 b2)
{
    if (a0 != b0) return a0 < b0;
    if (a1 != b1) return a1 < b1;
    return a2 < b2;
}

// scalar search energy in score units: s0 + floor(s1/1e6) + floor(s2/1e9)
__device__ __forceinline__ i64 rp_energy(i64 s0, i64 s1, i64 s2)
{
    return s0 + s1 / 1000000ll + s2 / 1000000000ll;
}

// Random part of the Metropolis test for an energy increase dE > 0:
// accept iff dE < (((tau * nl2(x)) >> 32) * max(e_old, SC)) >> 32, saturating to "accept".
__device__ __forceinline__ bool rp_accept_uphill(i64 e_old, i64 dE, i64 SC, u64 tau, u32 x)
{
    u64 nl = rp_nl2(x);
    u64 hi = __umul64hi(tau, nl), lo = tau * nl;
    if (hi >> 30) return true;                       // threshold >= 2^62
    u64 thr = (hi << 32) | (lo >> 32);
    u64 M = (u64)(e_old > SC ? e_old : SC);
    u64 bh = __umul64hi(thr, M), bl = thr * M;
    if (bh >> 31) return true;                       // bound >= 2^63
    u64 bound = (bh << 32) | (bl >> 32);
    return (u64)dE < bound;
}

#endif  // __CUDACC__
