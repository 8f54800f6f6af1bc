// C-ABI entry points of the RoutePack B200 library: argument checks, device memory
// ownership, kernel sequencing.  All arithmetic of the method runs in the kernels.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "rp_common.cuh"

thread_local int g_rp_last_cuda_error = 0;
long long g_rp_launches = 0;      // kernels launched by this library in this process

extern "C" int64_t rp_debug_launch_count(void) { return g_rp_launches; }

extern "C" int rp_last_cuda_error(void) { return g_rp_last_cuda_error; }

extern "C" const char *rp_strerror(int s)
{
    switch (s) {
        case RP_OK: return "ok";
        case RP_ERR_ARG: return "bad argument";
        case RP_ERR_SHAPE: return "inconsistent shapes";
        case RP_ERR_CONSERVATION: return "window fails the input checks (length range, negative count, or sum_e a != k*t)";
        case RP_ERR_INFEASIBLE: return "no feasible row count";
        case RP_ERR_RANGE: return "fixed-point range or on-chip memory budget exceeded";
        case RP_ERR_CUDA: return "CUDA error";
        case RP_ERR_STATE: return "call out of order";
        case RP_ERR_TIMEOUT: return "device-side wait timed out";
        case RP_ERR_INVALID_PLAN: return "incumbent failed validation";
        default: return "unknown status";
    }
}

// Device memory comes from one stream-ordered pool per device that keeps freed blocks cached
// (release threshold = unlimited), so that planning window after window does not pay for
// cudaMalloc/cudaFree; rp_release_cached_memory() hands the cache back to the driver.
#define RP_MAX_DEVICES 64
static cudaMemPool_t g_pools[RP_MAX_DEVICES];
static bool g_pool_ready[RP_MAX_DEVICES];

int rp_get_pool(int device, cudaMemPool_t *out)
{
    if (device < 0 || device >= RP_MAX_DEVICES) return RP_ERR_ARG;
    if (!g_pool_ready[device]) {
        cudaMemPoolProps props;
        memset(&props, 0, sizeof props);
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        RP_CUDA(cudaMemPoolCreate(&g_pools[device], &props));
        unsigned long long keep = ~0ull;
        RP_CUDA(cudaMemPoolSetAttribute(g_pools[device], cudaMemPoolAttrReleaseThreshold, &keep));
        g_pool_ready[device] = true;
    }
    *out = g_pools[device];
    return RP_OK;
}

extern "C" int rp_release_cached_memory(void)
{
    for (int d = 0; d < RP_MAX_DEVICES; ++d)
        if (g_pool_ready[d]) RP_CUDA(cudaMemPoolTrimTo(g_pools[d], 0));
    return RP_OK;
}

// Pinned staging blocks (512 bytes) for reading scalars back without a synchronous pageable copy;
// recycled across contexts because pinning memory is slow.
#include <mutex>
#include <vector>
static std::mutex g_pin_mutex;
static std::vector<void *> g_pin_free;
static void *pin_take()
{
    {
        std::lock_guard<std::mutex> lk(g_pin_mutex);
        if (!g_pin_free.empty()) { void *p = g_pin_free.back(); g_pin_free.pop_back(); return p; }
    }
    void *p = nullptr;
    if (cudaHostAlloc(&p, 512, cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
}
static void pin_give(void *p)
{
    if (!p) return;
    std::lock_guard<std::mutex> lk(g_pin_mutex);
    g_pin_free.push_back(p);
}

// A side stream with two events, recycled across contexts of a device like the pinned blocks:
// packing needs only the lengths, so it runs beside the check / placement / projection kernels.
struct RpSide { int device; cudaStream_t stream; cudaEvent_t fork, join; };
static std::vector<RpSide *> g_side_free;
static RpSide *side_take(int device)
{
    {
        std::lock_guard<std::mutex> lk(g_pin_mutex);
        for (size_t x = 0; x < g_side_free.size(); ++x)
            if (g_side_free[x]->device == device) {
                RpSide *s = g_side_free[x];
                g_side_free.erase(g_side_free.begin() + x);
                return s;
            }
    }
    RpSide *s = new RpSide;
    s->device = device;
    if (cudaStreamCreateWithFlags(&s->stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        delete s;
        return nullptr;
    }
    return s;
}
static void side_give(RpSide *s)
{
    if (!s) return;
    std::lock_guard<std::mutex> lk(g_pin_mutex);
    g_side_free.push_back(s);
}


// Optional stage timing: one flag for the process (a context only exists once rp_window_load has
// already queued the front end), events per context.
static int g_stage_timing = 0;
static void stage_mark(rp_ctx *c, int which, cudaStream_t stream)
{
    if (!c->ev_stage[0]) return;
    if (cudaEventRecord(c->ev_stage[which], stream) == cudaSuccess) c->ev_recorded |= 1u << which;
    else cudaGetLastError();
}

static bool is_device_ptr(const void *p)
{
    cudaPointerAttributes at;
    cudaError_t e = cudaPointerGetAttributes(&at, p);
    if (e != cudaSuccess) { cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

static int copy_out(rp_ctx *c, void *dst, const void *src, size_t bytes)
{
    if (!dst || !bytes) return RP_OK;
    RP_CUDA(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDefault, c->stream));
    return RP_OK;
}

static void free_population(rp_ctx *c)
{
    dev_free(c, c->d_pop_slab); c->d_pop_slab = nullptr;           // every buffer below is a piece of it
    c->buf[0].blob = nullptr; c->buf[1].blob = nullptr;
    c->d_W = nullptr; c->d_wloc = nullptr; c->d_wloc_next = nullptr; c->d_le_scratch = nullptr;
    c->d_wref = nullptr; c->d_wcount = nullptr; c->d_wfree = nullptr; c->d_wfree_head = nullptr;
    c->d_cand_layout = nullptr; c->d_inc_slot = nullptr;
    c->d_sync = nullptr;
    c->d_anc = nullptr; c->d_anc_next = nullptr; c->d_done = nullptr; c->d_term = nullptr; c->d_best = nullptr; c->d_best_step = nullptr;
    c->d_best_nlog = nullptr; c->d_digest = nullptr; c->d_F = nullptr;
    dev_free(c, c->d_sel_dist); c->d_sel_dist = nullptr;
    dev_free(c, c->d_log); c->d_log = nullptr;
    c->log_cap = 0;
}

static void free_trace(rp_ctx *c)
{
    dev_free(c, c->d_tr_term); dev_free(c, c->d_tr_best); dev_free(c, c->d_tr_inc);
    dev_free(c, c->d_tr_best_step); dev_free(c, c->d_tr_anc); dev_free(c, c->d_tr_digest);
    c->d_tr_term = c->d_tr_best = c->d_tr_inc = nullptr;
    c->d_tr_best_step = c->d_tr_anc = nullptr;
    c->d_tr_digest = nullptr;
    c->trace_levels = 0;
}

static void free_eval(rp_ctx *c)
{
    dev_free(c, c->d_eval_score); dev_free(c, c->d_eval_f64); dev_free(c, c->d_eval_W);
    dev_free(c, c->d_eval_cells); dev_free(c, c->d_eval_Esum); dev_free(c, c->d_eval_tickets);
    c->d_eval_score = nullptr; c->d_eval_f64 = nullptr; c->d_eval_W = nullptr;
    c->d_eval_cells = nullptr; c->d_eval_Esum = nullptr; c->d_eval_tickets = nullptr;
    c->eval_cap = 0; c->eval_W_n = 0;
}

extern "C" void rp_destroy(rp_ctx *c)
{
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    free_population(c); free_trace(c); free_eval(c);
    dev_free(c, c->own_t); dev_free(c, c->own_a); dev_free(c, c->d_load_slab); dev_free(c, c->d_static); dev_free(c, c->d_levels);
    pin_give(c->h_pin);
    for (int x = 0; x < RP_STAGE_EVENTS; ++x) if (c->ev_stage[x]) cudaEventDestroy(c->ev_stage[x]);
    side_give((RpSide *)c->side);
    free(c->h_levels);
    free(c);
}

static int reset_status(rp_ctx *c)
{
    RP_CUDA(cudaMemsetAsync(c->d_status, 0, sizeof(int) * RP_SW_COUNT, c->stream));
    return RP_OK;
}

static int read_status(rp_ctx *c, int out[RP_SW_COUNT])
{
    int *stage = (int *)(c->h_pin + 56);
    RP_CUDA(cudaMemcpyAsync(stage, c->d_status, sizeof(int) * RP_SW_COUNT, cudaMemcpyDeviceToHost, c->stream));
    RP_CUDA(cudaStreamSynchronize(c->stream));
    memcpy(out, stage, sizeof(int) * RP_SW_COUNT);
    return RP_OK;
}

static int window_load_impl(rp_ctx *c, const rp_config *cfg, const int32_t *lengths, const int32_t *demand)
{
    RpDims &dm = c->dm;
    const int N = cfg->n_samples, L = cfg->n_layers, E = cfg->n_experts, D = cfg->dp_width, P = cfg->ep_width;
    // EDP partition
    int *edp = (int *)malloc(sizeof(int) * D);
    int G = 0;
    for (int d = 0; d < D; ++d) {
        edp[d] = cfg->edp_of_dp ? cfg->edp_of_dp[d] : d;
        if (edp[d] < 0 || edp[d] >= D) { free(edp); return RP_ERR_SHAPE; }
        if (edp[d] + 1 > G) G = edp[d] + 1;
    }
    int *off = (int *)calloc(G + 1, sizeof(int)), *list = (int *)malloc(sizeof(int) * D);
    for (int d = 0; d < D; ++d) off[edp[d] + 1]++;
    int maxshard = 0;
    for (int g = 0; g < G; ++g) {
        if (off[g + 1] == 0) { free(edp); free(off); free(list); return RP_ERR_SHAPE; }   // unused shard id
        if (off[g + 1] > maxshard) maxshard = off[g + 1];
        off[g + 1] += off[g];
    }
    {
        int *cursor = (int *)malloc(sizeof(int) * G);
        for (int g = 0; g < G; ++g) cursor[g] = off[g];
        for (int d = 0; d < D; ++d) list[cursor[edp[d]]++] = d;
        free(cursor);
    }
    dm.N = N; dm.L = L; dm.E = E; dm.k = cfg->top_k; dm.C = cfg->token_cap; dm.D = D; dm.P = P; dm.G = G;
    dm.H = E / P; dm.S = cfg->n_stages;
    dm.R = 0; dm.K = 0; dm.RG = 0; dm.LP = L * P; dm.slices = 0;
    dm.asum = 0; dm.bsum = 0;
    for (int s = 0; s < RP_MAX_STAGES; ++s) { dm.ahat[s] = 0; dm.bhat[s] = 0; }
    for (int s = 0; s < dm.S; ++s) {
        dm.ahat[s] = (i64)floor(cfg->alpha[s] * 256.0 + 0.5);
        dm.bhat[s] = (i64)floor(cfg->beta[s] * 256.0 + 0.5);
        dm.asum += dm.ahat[s]; dm.bsum += dm.bhat[s];
    }
    dm.SC = ((i64)dm.C * dm.C) << RP_FBITS;
    dm.EC = (i64)dm.C << RP_FBITS;
    // rank loads must fit int32: W <= k * C * |D_g|
    if ((double)dm.k * dm.C * maxshard >= 2147483648.0) { free(edp); free(off); free(list); return RP_ERR_RANGE; }

    // inputs: adopt device arrays, copy host arrays
    const size_t n_a = (size_t)N * L * E;
    int st = RP_OK;
    do {
        if (is_device_ptr(lengths)) c->d_t = lengths;
        else {
            if ((st = dev_alloc(c, &c->own_t, N)) != RP_OK) break;
            if (cudaMemcpyAsync(c->own_t, lengths, sizeof(int) * N, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) { st = RP_ERR_CUDA; break; }
            c->d_t = c->own_t;
        }
        if (is_device_ptr(demand)) c->d_a = demand;
        else {
            if ((st = dev_alloc(c, &c->own_a, n_a)) != RP_OK) break;
            if (cudaMemcpyAsync(c->own_a, demand, sizeof(int) * n_a, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) { st = RP_ERR_CUDA; break; }
            c->d_a = c->own_a;
        }
        // everything sized by the window alone comes out of one allocation
        int n_pow2 = 1;
        while (n_pow2 < N) n_pow2 <<= 1;
        const size_t n_tab = (size_t)2 * D + G + 1;
        RpSlab slab = { nullptr, 0 };
        for (int pass = 0; pass < 2 && st == RP_OK; ++pass) {
            slab.off = 0;
            slab.take(&c->d_Lagg, (size_t)L * E);
            slab.take(&c->d_status, RP_SW_COUNT);
            slab.take(&c->d_counters, 8);
            slab.take(&c->d_edp, n_tab);
            slab.take(&c->d_pi, (size_t)L * E);
            slab.take(&c->d_inv, (size_t)L * E);
            slab.take(&c->d_rank_load, (size_t)L * P);
            slab.take(&c->d_q, (size_t)N * L * P);
            slab.take(&c->d_sort_keys, (size_t)2 * n_pow2);
            slab.take(&c->d_seed_layout, N);
            slab.take(&c->d_order, N);
            slab.take(&c->d_pack_out, 4);
            slab.take(&c->d_inc_layout, N);
            slab.take(&c->d_inc_score, 3);
            slab.take(&c->d_seed_score, 3);
            slab.take(&c->d_best_score, 3);
            slab.take(&c->d_best_f64, 3);
            if (pass == 0) { st = dev_alloc(c, &c->d_load_slab, slab.off); slab.base = c->d_load_slab; }
        }
        if (st != RP_OK) break;
        c->d_dp_list = c->d_edp + D;
        c->d_dp_off = c->d_dp_list + D;
        // input checks + aggregate expert load + token total in one pass over the demand tensor,
        // put in flight before the rest of the set-up
        if (cudaMemsetAsync(c->d_counters, 0, sizeof(i64) * 8, c->stream) != cudaSuccess) { st = RP_ERR_CUDA; break; }
        if ((st = reset_status(c)) != RP_OK) break;
        stage_mark(c, RP_EV_K1_0, c->stream);
        if ((st = rp_launch_check_reduce(c)) != RP_OK) break;
        stage_mark(c, RP_EV_K1_1, c->stream);
        // the EDP tables: one copy (pageable source: staged before the call returns)
        int *tab = (int *)malloc(sizeof(int) * n_tab);
        memcpy(tab, edp, sizeof(int) * D);
        memcpy(tab + D, list, sizeof(int) * D);
        memcpy(tab + 2 * D, off, sizeof(int) * (G + 1));
        const cudaError_t e = cudaMemcpyAsync(c->d_edp, tab, sizeof(int) * n_tab, cudaMemcpyHostToDevice, c->stream);
        free(tab);
        if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; st = RP_ERR_CUDA; break; }
    } while (0);
    free(edp); free(off); free(list);
    RP_TRY(st);

    // Placement, projection and packing depend on nothing but the inputs: they are queued right
    // behind the checks, so that the GPU works on them while the host waits for the verdict
    // (rp_place_experts and rp_pack_rows then only hand the results over).
    // Packing reads only the lengths: it goes to a side stream that forks here and joins before the
    // row count is read back.
    RpSide *side = (RpSide *)c->side;
    bool forked = false;
    if (side && cudaEventRecord(side->fork, c->stream) == cudaSuccess &&
        cudaStreamWaitEvent(side->stream, side->fork, 0) == cudaSuccess) {
        stage_mark(c, RP_EV_PACK_0, side->stream);
        c->eager_pack = (rp_launch_pack_on(c, side->stream) == RP_OK);
        stage_mark(c, RP_EV_PACK_1, side->stream);
        forked = (cudaEventRecord(side->join, side->stream) == cudaSuccess);
        if (!forked) { cudaStreamSynchronize(side->stream); c->eager_pack = 0; }
    }
    stage_mark(c, RP_EV_K2_0, c->stream);
    c->eager_place = (rp_launch_lpt(c) == RP_OK);
    stage_mark(c, RP_EV_K2_1, c->stream);
    c->eager_place = c->eager_place && (rp_launch_project(c) == RP_OK);
    stage_mark(c, RP_EV_K3_1, c->stream);
    if (forked) RP_CUDA(cudaStreamWaitEvent(c->stream, side->join, 0));
    else c->eager_pack = (rp_launch_pack(c, 0) == RP_OK);
    if (c->eager_pack)
        RP_CUDA(cudaMemcpyAsync(c->h_pin + 10, c->d_pack_out, sizeof(int) * 4, cudaMemcpyDeviceToHost, c->stream));

    // verdict of the checks and the token total ride back in the pinned block
    RP_CUDA(cudaMemcpyAsync(c->h_pin + 8, c->d_counters + 7, sizeof(i64), cudaMemcpyDeviceToHost, c->stream));
    int sw[RP_SW_COUNT];
    RP_TRY(read_status(c, sw));
    if (sw[RP_SW_BAD_SAMPLE]) return RP_ERR_CONSERVATION;
    memcpy(c->pack_out, c->h_pin + 10, sizeof(int) * 4);

    // fixed-point range of the score: s1 <= (2^8*C*L*k + (asum+bsum)*C) * sum t  must stay below 2^62
    const double total = (double)c->h_pin[8];
    double bound = ((double)dm.EC * L * dm.k + (double)(dm.asum + dm.bsum) * dm.C) * total;
    if (bound >= 4.0e18) return RP_ERR_RANGE;
    return RP_OK;
}

extern "C" int rp_window_load(rp_ctx **out, const rp_config *cfg, const int32_t *lengths,
                              const int32_t *demand, void *cuda_stream)
{
    if (!out) return RP_ERR_ARG;
    *out = nullptr;
    if (!cfg || !lengths || !demand) return RP_ERR_ARG;
    if (cfg->n_samples < 1 || cfg->n_layers < 1 || cfg->n_experts < 1 || cfg->top_k < 1 || cfg->token_cap < 1 ||
        cfg->dp_width < 1 || cfg->ep_width < 1 || cfg->pop_size < 1 || cfg->min_rows < 0)
        return RP_ERR_ARG;
    if (cfg->n_stages < 1 || cfg->n_stages > RP_MAX_STAGES || !cfg->alpha || !cfg->beta) return RP_ERR_ARG;
    for (int s = 0; s < cfg->n_stages; ++s)
        if (!(cfg->alpha[s] >= 0.0) || !(cfg->beta[s] >= 0.0) || cfg->alpha[s] > 1e6 || cfg->beta[s] > 1e6) return RP_ERR_ARG;
    if (cfg->n_experts % cfg->ep_width != 0 || cfg->n_samples < cfg->dp_width) return RP_ERR_SHAPE;
    if (cfg->ep_width > RP_MAX_EP || cfg->dp_width > 4096 || cfg->n_experts > 1024) return RP_ERR_RANGE;
    if (cfg->token_cap > (1 << 24) || cfg->n_samples > (1 << 20) || cfg->pop_size > (1 << 20)) return RP_ERR_RANGE;
    if ((long long)cfg->n_layers * cfg->ep_width > (1 << 20)) return RP_ERR_RANGE;

    rp_ctx *c = (rp_ctx *)calloc(1, sizeof(rp_ctx));
    if (!c) return RP_ERR_ARG;
    if (cudaGetDevice(&c->device) != cudaSuccess) { free(c); return RP_ERR_CUDA; }
    c->stream = (cudaStream_t)cuda_stream;
    c->cfg = *cfg;
    c->cfg.edp_of_dp = nullptr; c->cfg.alpha = nullptr; c->cfg.beta = nullptr;
    c->Ppop = cfg->pop_size;
    c->h_pin = (i64 *)pin_take();
    if (!c->h_pin) { free(c); return RP_ERR_CUDA; }
    c->side = side_take(c->device);          // optional: without it everything runs on the one stream
    if (g_stage_timing)
        for (int x = 0; x < RP_STAGE_EVENTS; ++x)
            if (cudaEventCreate(&c->ev_stage[x]) != cudaSuccess) { cudaGetLastError(); c->ev_stage[0] = nullptr; break; }
    int st = window_load_impl(c, cfg, lengths, demand);
    if (st != RP_OK) { rp_destroy(c); return st; }
    c->stage = 1;
    *out = c;
    return RP_OK;
}

extern "C" int rp_place_experts(rp_ctx *c, int32_t *pi, int64_t *rank_load)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage < 1) return RP_ERR_STATE;
    const RpDims &dm = c->dm;
    if (!c->eager_place) {
        RP_TRY(rp_launch_lpt(c));
        RP_TRY(rp_launch_project(c));
    }
    c->eager_place = 0;               // a repeated call recomputes
    RP_TRY(copy_out(c, pi, c->d_pi, sizeof(int) * (size_t)dm.L * dm.E));
    RP_TRY(copy_out(c, rank_load, c->d_rank_load, sizeof(i64) * (size_t)dm.L * dm.P));
    // Outputs are complete when the call returns (nothing to wait for when none was asked for).
    if (pi || rank_load) RP_CUDA(cudaStreamSynchronize(c->stream));
    if (c->stage < 2) c->stage = 2;
    return RP_OK;
}

static int ensure_eval_scratch(rp_ctx *c, size_t n, bool want_W)
{
    const RpDims &dm = c->dm;
    if (n > c->eval_cap) {
        dev_free(c, c->d_eval_score); dev_free(c, c->d_eval_f64); dev_free(c, c->d_eval_cells);
        dev_free(c, c->d_eval_Esum); dev_free(c, c->d_eval_tickets);
        c->d_eval_score = nullptr; c->d_eval_f64 = nullptr; c->d_eval_cells = nullptr;
        c->d_eval_Esum = nullptr; c->d_eval_tickets = nullptr;
        c->eval_cap = 0;
        RP_TRY(dev_alloc(c, &c->d_eval_score, n * 3));
        RP_TRY(dev_alloc(c, &c->d_eval_f64, n * 3));
        RP_TRY(dev_alloc(c, &c->d_eval_cells, n * dm.N));
        RP_TRY(dev_alloc(c, &c->d_eval_Esum, n * dm.RG));
        RP_TRY(dev_alloc(c, &c->d_eval_tickets, n));
        RP_CUDA(cudaMemsetAsync(c->d_eval_tickets, 0, sizeof(int) * n, c->stream));
        c->eval_cap = n;
    }
    if (want_W && (int)n > c->eval_W_n) {
        dev_free(c, c->d_eval_W);
        c->d_eval_W = nullptr; c->eval_W_n = 0;
        RP_TRY(dev_alloc(c, &c->d_eval_W, n * dm.RG * dm.LP));
        c->eval_W_n = (int)n;
    }
    return RP_OK;
}

__global__ void k_iota(int *out, int n, int first)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x < n) out[x] = first + x;
}

// Population bookkeeping of a fresh seed in one launch: every member descends from slot 0, whose
// rank loads sit in cell 0 and are copied into a cell of the member's own (P + m) at level 0; the
// seed is the incumbent.
__global__ void k_init_population(int P, int N, int *__restrict__ anc, int *__restrict__ wloc, int *__restrict__ wloc_next,
                                  int *__restrict__ done, const int *__restrict__ seed_layout, int *__restrict__ inc_layout,
                                  const i64 *__restrict__ inc_score, i64 *__restrict__ seed_score)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x < P) { anc[x] = 0; wloc[x] = 0; wloc_next[x] = P + x; }
    if (x < N) inc_layout[x] = seed_layout[x];
    if (x < 3) seed_score[x] = inc_score[x];
    if (x == 0) *done = 0;
}

static int build_population(rp_ctx *c);

extern "C" int rp_pack_rows(rp_ctx *c, int32_t *n_rows, int32_t *certified)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage < 2) return RP_ERR_STATE;
    RpDims &dm = c->dm;
    c->best_ready = 0;
    int *po = c->pack_out;
    if (!c->eager_pack) {
        RP_TRY(rp_launch_pack(c, 0));
        RP_CUDA(cudaMemcpyAsync(c->h_pin + 10, c->d_pack_out, sizeof(int) * 4, cudaMemcpyDeviceToHost, c->stream));
        RP_CUDA(cudaStreamSynchronize(c->stream));
        memcpy(c->pack_out, c->h_pin + 10, sizeof(int) * 4);
    }
    c->eager_pack = 0;                // a repeated call recomputes
    if (po[3] || po[0] <= 0) return RP_ERR_INFEASIBLE;
    c->Rstar = po[0]; c->certified = po[1];
    dm.R = po[0]; dm.K = dm.R * dm.D; dm.RG = dm.R * dm.G;
    if (dm.K > 65535) return RP_ERR_RANGE;
    RP_TRY(build_population(c));
    if (n_rows) *n_rows = c->Rstar;
    if (certified) *certified = c->certified;
    c->stage = 3;
    return RP_OK;
}

// Buffers of a population of c->Ppop members for the row count in c->dm, every member a copy of the
// length-only seed (evaluated once into slot 0, which all slots descend from); the seed is the incumbent.
static int build_population(rp_ctx *c)
{
    RpDims &dm = c->dm;
    rp_decide_layouts(c);
    int nt; size_t smem;
    rp_anneal_smem_bytes(c, &nt, &smem);
    if (smem > 220 * 1024) return RP_ERR_RANGE;

    // population buffers
    free_population(c); free_eval(c);
    const size_t P = (size_t)c->Ppop, wn = (size_t)dm.RG * dm.LP;
    {
        RpSlab slab = { nullptr, 0 };
        for (int pass = 0; pass < 2; ++pass) {
            slab.off = 0;
            slab.take(&c->buf[0].blob, P * (size_t)c->bl.bytes);
            slab.take(&c->buf[1].blob, P * (size_t)c->bl.bytes);
            slab.take(&c->d_W, 2 * P * wn);
            slab.take(&c->d_wloc, P);
            slab.take(&c->d_wloc_next, P);
            slab.take(&c->d_le_scratch, 6 * P);
            if (rp_uses_slices(c->dm)) {
                slab.take(&c->d_wref, 2 * P * (size_t)dm.RG);
                slab.take(&c->d_wcount, 2 * P * (size_t)dm.RG);
                slab.take(&c->d_wfree, 2 * P * (size_t)dm.RG);
                slab.take(&c->d_wfree_head, 2);
            }
            slab.take(&c->d_inc_slot, 1);
            if (rp_uses_wpc(c->dm)) slab.take(&c->d_cand_layout, P * (size_t)c->dm.N);
            slab.take(&c->d_anc, P);
            slab.take(&c->d_anc_next, P);
            slab.take(&c->d_done, 1);
            slab.take(&c->d_sync, P + 1);                // arrival counter, then one state-complete flag per member
            slab.take(&c->d_term, 2 * P * 3);            // reports: two sets, taken in turn by the launch that runs all levels
            slab.take(&c->d_best, 2 * P * 3);
            slab.take(&c->d_best_step, 2 * P);
            slab.take(&c->d_best_nlog, 2 * P);
            slab.take(&c->d_digest, 2 * P);
            slab.take(&c->d_F, P);
            if (pass == 0) { RP_TRY(dev_alloc(c, &c->d_pop_slab, slab.off)); slab.base = c->d_pop_slab; }
        }
    }
    c->cur = 0;
    if (c->d_wcount) RP_CUDA(cudaMemsetAsync(c->d_wcount, 0, sizeof(int) * 2 * P * (size_t)dm.RG, c->stream));
    // every member starts as the length-only seed: evaluate it once into slot 0 and let all
    // slots descend from slot 0
    dev_free(c, c->d_static); c->d_static = nullptr;
    RP_TRY(dev_alloc(c, &c->d_static, (size_t)c->sl.bytes));
    stage_mark(c, RP_EV_SEED_0, c->stream);
    RP_TRY(rp_launch_build_static(c));
    RP_TRY(ensure_eval_scratch(c, 1, false));
    RP_TRY(rp_launch_cells_from_layouts(c, c->d_seed_layout, 1, c->d_eval_cells));
    RP_TRY(rp_launch_eval(c, c->d_eval_cells, 1, c->d_W, c->buf[0].blob, c->d_inc_score, nullptr));
    {
        const size_t n = P > (size_t)dm.N ? P : (size_t)dm.N;
        k_init_population<<<(int)((n + 255) / 256), 256, 0, c->stream>>>((int)P, dm.N, c->d_anc, c->d_wloc, c->d_wloc_next, c->d_done,
                                                                          c->d_seed_layout, c->d_inc_layout, c->d_inc_score,
                                                                          c->d_seed_score);
        ++g_rp_launches;
        RP_CUDA(cudaGetLastError());
    }
    stage_mark(c, RP_EV_SEED_1, c->stream);
    return RP_OK;
}

__global__ void k_gather_cells(const char *__restrict__ blobs, RpBlob bl, const int *__restrict__ anc, int N,
                               unsigned short *__restrict__ dst16, int *__restrict__ dst32)
{
    const int j = blockIdx.x;
    const unsigned short *s = (const unsigned short *)(blobs + (size_t)anc[j] * bl.bytes + bl.off_cell);
    for (int i = threadIdx.x; i < N; i += blockDim.x) {
        if (dst16) dst16[(size_t)j * N + i] = s[i];
        if (dst32) dst32[(size_t)j * N + i] = s[i];
    }
}

extern "C" int rp_eval_population(rp_ctx *c, const int32_t *layouts, int32_t n, int64_t *score_fx, double *score_f64)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    const RpDims &dm = c->dm;
    if (!layouts) n = c->Ppop;
    if (n < 1) return RP_ERR_ARG;
    const bool keepW = layouts && n <= 64;
    RP_TRY(ensure_eval_scratch(c, (size_t)n, keepW));
    if (layouts) {
        const int *dl = layouts;
        int *tmp = nullptr;
        if (!is_device_ptr(layouts)) {
            RP_TRY(dev_alloc(c, &tmp, (size_t)n * dm.N));
            cudaError_t e = cudaMemcpyAsync(tmp, layouts, sizeof(int) * (size_t)n * dm.N, cudaMemcpyHostToDevice, c->stream);
            if (e != cudaSuccess) { dev_free(c, tmp); g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
            dl = tmp;
        }
        RP_TRY(reset_status(c));
        int st = rp_launch_cells_from_layouts(c, dl, n, c->d_eval_cells);
        int sw[RP_SW_COUNT];
        if (st == RP_OK) st = read_status(c, sw);
        dev_free(c, tmp);
        RP_TRY(st);
        if (sw[RP_SW_BAD_LAYOUT]) return RP_ERR_ARG;
    } else {
        k_gather_cells<<<n, 256, 0, c->stream>>>(c->buf[c->cur].blob, c->bl, c->d_anc, dm.N, c->d_eval_cells, nullptr);
        ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    }
    RP_TRY(rp_launch_eval(c, c->d_eval_cells, n, keepW ? c->d_eval_W : nullptr, nullptr, c->d_eval_score,
                          c->d_eval_f64));
    RP_TRY(copy_out(c, score_fx, c->d_eval_score, sizeof(i64) * 3 * (size_t)n));
    RP_TRY(copy_out(c, score_f64, c->d_eval_f64, sizeof(double) * 3 * (size_t)n));
    RP_CUDA(cudaStreamSynchronize(c->stream));
    return RP_OK;
}

// Randomized fixed-row seeds (Algorithm 2, trial loop): member 0 keeps the length-only seed, every
// other member runs its own WindowShuffle + RandomizedBestFit trial; all members are then scored
// from scratch and the incumbent becomes the best of them.
// Scores `lay` [P_pop][N] from scratch, makes it the population (member m owns rank-load cell m)
// and makes the best member the incumbent (lowest index on ties).
// Members n_distinct, n_distinct + 1, ... repeat the first n_distinct layouts in turn: member m descends
// from member m mod n_distinct (whose state it reads when the first level starts) and works in a
// rank-load cell of the other half, as the members of a freshly built population do.
__global__ void k_descend_cyclic(int P, int nd, int *__restrict__ anc, int *__restrict__ wloc, int *__restrict__ wloc_next)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m < P) { anc[m] = m % nd; wloc[m] = m % nd; wloc_next[m] = P + m; }
}

// n_distinct > 0: rows n_distinct .. P_pop-1 of `lay` repeat the first n_distinct rows cyclically, so
// only those are scored and every other member descends from its original (no state is copied).
static int install_population(rp_ctx *c, const int *lay, int n_distinct = 0)
{
    const size_t P = (size_t)c->Ppop;
    const size_t ne = (n_distinct > 0 && (size_t)n_distinct < P) ? (size_t)n_distinct : P;
    c->best_ready = 0;
    i64 *best = nullptr;
    RP_TRY(dev_alloc(c, &best, 3));
    int st = ensure_eval_scratch(c, ne, false);
    if (st == RP_OK) st = rp_launch_cells_from_layouts(c, lay, (int)ne, c->d_eval_cells);
    c->cur = 0;
    if (st == RP_OK) st = rp_launch_eval(c, c->d_eval_cells, (int)ne, c->d_W, c->buf[0].blob, c->d_eval_score, nullptr);
    if (st == RP_OK && ne == P) {
        k_iota<<<(int)((P + 255) / 256), 256, 0, c->stream>>>(c->d_wloc, (int)P, 0);
        k_iota<<<(int)((P + 255) / 256), 256, 0, c->stream>>>(c->d_wloc_next, (int)P, 0);
        k_iota<<<(int)((P + 255) / 256), 256, 0, c->stream>>>(c->d_anc, (int)P, 0);
        g_rp_launches += 3;
    } else if (st == RP_OK) {
        k_descend_cyclic<<<(int)((P + 255) / 256), 256, 0, c->stream>>>((int)P, (int)ne, c->d_anc, c->d_wloc, c->d_wloc_next);
        ++g_rp_launches;
    }
    if (st == RP_OK) st = rp_launch_pick_best(c, c->d_eval_score, lay, (int)ne, best);
    cudaError_t e = cudaSuccess;
    if (st == RP_OK) e = cudaMemcpyAsync(c->d_seed_score, best, sizeof(i64) * 3, cudaMemcpyDeviceToDevice, c->stream);
    dev_free(c, best);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return st;
}

extern "C" int rp_seed_population(rp_ctx *c, int32_t choice_width, int32_t *n_own)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage != 3) return RP_ERR_STATE;          // after rp_pack_rows, before rp_anneal
    if (choice_width < 1 || choice_width > 32) return RP_ERR_ARG;
    const RpDims &dm = c->dm;
    if (dm.K > 2048) return RP_ERR_RANGE;            // per-warp cell tables live in shared memory
    const size_t P = (size_t)c->Ppop;
    int *lay = nullptr, *ok = nullptr;
    RP_TRY(dev_alloc(c, &lay, P * dm.N));
    int st = dev_alloc(c, &ok, P);
    if (st == RP_OK) st = rp_launch_seed_trials(c, choice_width, lay, ok);
    if (st == RP_OK) st = install_population(c, lay);
    int *h_ok = (int *)malloc(sizeof(int) * P);
    cudaError_t e = cudaSuccess;
    if (st == RP_OK) {
        e = cudaMemcpyAsync(h_ok, ok, sizeof(int) * P, cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    }
    int own = 0;
    if (st == RP_OK && e == cudaSuccess) for (size_t j = 0; j < P; ++j) own += h_ok[j];
    free(h_ok);
    dev_free(c, lay); dev_free(c, ok);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    RP_TRY(st);
    if (n_own) *n_own = own;
    return RP_OK;
}

__global__ void k_count_changed(const int *__restrict__ a, const int *__restrict__ b, int N, int *__restrict__ out)
{
    __shared__ int diff;
    if (threadIdx.x == 0) diff = 0;
    __syncthreads();
    int d = 0;
    for (int i = threadIdx.x; i < N; i += blockDim.x) d |= (a[(size_t)blockIdx.x * N + i] != b[(size_t)blockIdx.x * N + i]);
    if (d) diff = 1;
    __syncthreads();
    if (threadIdx.x == 0 && diff) atomicAdd(out, 1);
}

extern "C" int rp_pair_population(rp_ctx *c, int32_t choice_width, int32_t *n_changed)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage != 3) return RP_ERR_STATE;          // after rp_pack_rows, before rp_anneal
    if (choice_width < 1 || choice_width > 32) return RP_ERR_ARG;
    const RpDims &dm = c->dm;
    const size_t P = (size_t)c->Ppop;
    int *lay = nullptr, *out = nullptr, *prof = nullptr, *cnt = nullptr;
    RP_TRY(dev_alloc(c, &lay, P * dm.N));
    int st = dev_alloc(c, &out, P * dm.N);
    if (st == RP_OK) st = dev_alloc(c, &cnt, 1);
    const int batch = (int)(P - 1 < 1024 ? P - 1 : 1024);          // members paired per launch (bounds the scratch)
    if (st == RP_OK && batch > 0) st = dev_alloc(c, &prof, (size_t)batch * dm.K * dm.LP);
    cudaError_t e = cudaSuccess;
    if (st == RP_OK) {
        k_gather_cells<<<c->Ppop, 256, 0, c->stream>>>(c->buf[c->cur].blob, c->bl, c->d_anc, dm.N, nullptr, lay);
        ++g_rp_launches;
        e = cudaMemcpyAsync(out, lay, sizeof(int) * dm.N, cudaMemcpyDeviceToDevice, c->stream);     // member 0 stays
        if (e == cudaSuccess) e = cudaMemsetAsync(cnt, 0, sizeof(int), c->stream);
    }
    for (int first = 1; st == RP_OK && e == cudaSuccess && first < (int)P; first += batch) {
        const int count = (int)P - first < batch ? (int)P - first : batch;
        st = rp_launch_edp_pair(c, lay, out, prof, first, count, choice_width);
    }
    if (st == RP_OK && e == cudaSuccess) {
        k_count_changed<<<c->Ppop, 256, 0, c->stream>>>(lay, out, dm.N, cnt);
        ++g_rp_launches;
        st = install_population(c, out);
    }
    int h_cnt = 0;
    if (st == RP_OK && e == cudaSuccess) {
        e = cudaMemcpyAsync(&h_cnt, cnt, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    }
    dev_free(c, lay); dev_free(c, out); dev_free(c, prof); dev_free(c, cnt);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    RP_TRY(st);
    if (n_changed) *n_changed = h_cnt;
    return RP_OK;
}

extern "C" int rp_select_population(rp_ctx *c, int32_t n_proj, int64_t eta_q16, int32_t *n_distinct, int32_t *order)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage != 3) return RP_ERR_STATE;          // after rp_pack_rows, before rp_anneal
    if (n_proj < 1 || n_proj > 64 || eta_q16 < 0 || eta_q16 > ((int64_t)1 << 40)) return RP_ERR_ARG;
    const RpDims &dm = c->dm;
    if ((double)dm.C * dm.C * dm.D * 65536.0 >= 9.0e18) return RP_ERR_RANGE;      // Q16 row feature of the squared lengths
    const size_t P = (size_t)c->Ppop;
    int *lay = nullptr, *out = nullptr, *d_order = nullptr, *d_nd = nullptr;
    dev_free(c, c->d_sel_dist); c->d_sel_dist = nullptr;
    RP_TRY(dev_alloc(c, &lay, P * dm.N));
    int st = dev_alloc(c, &out, P * dm.N);
    if (st == RP_OK) st = dev_alloc(c, &d_order, P);
    if (st == RP_OK) st = dev_alloc(c, &d_nd, 1);
    if (st == RP_OK) st = dev_alloc(c, &c->d_sel_dist, P * P);
    if (st == RP_OK) {
        k_gather_cells<<<c->Ppop, 256, 0, c->stream>>>(c->buf[c->cur].blob, c->bl, c->d_anc, dm.N, nullptr, lay);
        ++g_rp_launches;
        // exact scores of the members as they stand
        st = ensure_eval_scratch(c, P, false);
    }
    if (st == RP_OK) st = rp_launch_cells_from_layouts(c, lay, (int)P, c->d_eval_cells);
    if (st == RP_OK) st = rp_launch_eval(c, c->d_eval_cells, (int)P, nullptr, nullptr, c->d_eval_score, nullptr);
    if (st == RP_OK) st = rp_launch_select(c, lay, out, c->d_eval_score, n_proj, eta_q16, d_order, d_nd, c->d_sel_dist);
    if (st == RP_OK) st = install_population(c, out);
    int *h = (int *)malloc(sizeof(int) * (P + 1));
    cudaError_t e = cudaSuccess;
    if (st == RP_OK) {
        e = cudaMemcpyAsync(h, d_order, sizeof(int) * P, cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(h + P, d_nd, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    }
    if (st == RP_OK && e == cudaSuccess) {
        if (n_distinct) *n_distinct = h[P];
        if (order) memcpy(order, h, sizeof(int) * P);
    }
    free(h);
    dev_free(c, lay); dev_free(c, out); dev_free(c, d_order); dev_free(c, d_nd);
    if (!c->trace_on) { dev_free(c, c->d_sel_dist); c->d_sel_dist = nullptr; }      // kept for inspection only
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return st;
}

// Candidate 1 of Algorithm 2: the better of the length-only seed and its pairing (the seed on ties).
__global__ void k_keep_better_of_seed(const int *__restrict__ seed_layout, const i64 *__restrict__ seed_score,
                                      int *__restrict__ lay1, const i64 *__restrict__ score1, int N)
{
    const bool paired_wins = rp_lex_less(score1[0], score1[1], score1[2], seed_score[0], seed_score[1], seed_score[2]);
    if (paired_wins) return;
    for (int i = threadIdx.x; i < N; i += blockDim.x) lay1[i] = seed_layout[i];
}
__global__ void k_pick_rows(int N, const int *__restrict__ pick, const int *__restrict__ lay, int *__restrict__ out)
{
    const int *src = lay + (size_t)pick[blockIdx.x] * N;
    for (int i = threadIdx.x; i < N; i += blockDim.x) out[(size_t)blockIdx.x * N + i] = src[i];
}

// Algorithm 2 as one operation over M candidates: x_length, x_paired = min_Score{x_length,
// EDPAwarePair(x_length)}, M - 2 trials (WindowShuffle -> RandomizedBestFit -> EDPAwarePair),
// CanonicalMap over all of them and QualityDiversitySelect down to the population, repeated
// cyclically when fewer distinct plans exist.  The candidates are worked on as a population of M
// members of their own; the population proper is rebuilt from the selected ones afterwards.
extern "C" int rp_init_population(rp_ctx *c, int32_t n_candidates, int32_t choice_width, int32_t n_proj, int64_t eta_q16,
                                  int32_t *n_distinct, int32_t *picked)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage != 3) return RP_ERR_STATE;
    if (n_candidates < 2 || n_candidates > (1 << 16) || choice_width < 1 || choice_width > 32) return RP_ERR_ARG;
    if (n_proj < 1 || n_proj > 64 || eta_q16 < 0 || eta_q16 > ((int64_t)1 << 40)) return RP_ERR_ARG;
    const RpDims &dm = c->dm;
    if (dm.K > 2048) return RP_ERR_RANGE;
    if ((double)dm.C * dm.C * dm.D * 65536.0 >= 9.0e18) return RP_ERR_RANGE;
    const int P = c->Ppop, M = n_candidates;
    int *lay = nullptr, *out = nullptr, *sel = nullptr, *ok = nullptr, *prof = nullptr, *d_order = nullptr, *d_nd = nullptr;
    int *fin = nullptr, *d_pick = nullptr;
    i64 *dist = nullptr;
    int *h = (int *)malloc(sizeof(int) * ((size_t)M + 1 + P));
    int st = RP_OK;
    cudaError_t e = cudaSuccess;
    // the candidates as a population of their own
    c->Ppop = M;
    st = build_population(c);
    do {
        if (st != RP_OK) break;
        if ((st = dev_alloc(c, &lay, (size_t)M * dm.N)) != RP_OK) break;
        if ((st = dev_alloc(c, &out, (size_t)M * dm.N)) != RP_OK) break;
        if ((st = dev_alloc(c, &sel, (size_t)M * dm.N)) != RP_OK) break;
        if ((st = dev_alloc(c, &ok, M)) != RP_OK) break;
        if ((st = dev_alloc(c, &d_order, M)) != RP_OK) break;
        if ((st = dev_alloc(c, &d_nd, 1)) != RP_OK) break;
        if ((st = dev_alloc(c, &dist, (size_t)M * M)) != RP_OK) break;
        const int batch = M - 1 < 1024 ? M - 1 : 1024;
        if ((st = dev_alloc(c, &prof, (size_t)batch * dm.K * dm.LP)) != RP_OK) break;
        // trials 2 .. M-1; candidates 0 and 1 start as the length-only seed
        if ((st = rp_launch_seed_trials(c, choice_width, lay, ok)) != RP_OK) break;
        if ((e = cudaMemcpyAsync(lay + dm.N, c->d_seed_layout, sizeof(int) * dm.N, cudaMemcpyDeviceToDevice, c->stream)) != cudaSuccess) break;
        // pairing of every candidate but x_length
        if ((e = cudaMemcpyAsync(out, lay, sizeof(int) * dm.N, cudaMemcpyDeviceToDevice, c->stream)) != cudaSuccess) break;
        for (int first = 1; st == RP_OK && first < M; first += batch)
            st = rp_launch_edp_pair(c, lay, out, prof, first, M - first < batch ? M - first : batch, choice_width);
        if (st != RP_OK) break;
        // x_paired: the pairing of the seed only if it scores lower
        if ((st = ensure_eval_scratch(c, (size_t)M, false)) != RP_OK) break;
        if ((st = rp_launch_cells_from_layouts(c, out + dm.N, 1, c->d_eval_cells)) != RP_OK) break;
        if ((st = rp_launch_eval(c, c->d_eval_cells, 1, nullptr, nullptr, c->d_eval_score, nullptr)) != RP_OK) break;
        k_keep_better_of_seed<<<1, 256, 0, c->stream>>>(c->d_seed_layout, c->d_seed_score, out + dm.N, c->d_eval_score, dm.N);
        ++g_rp_launches;
        // all candidates scored and installed, then the selection over them
        if ((st = install_population(c, out)) != RP_OK) break;
        if ((st = rp_launch_select(c, out, sel, c->d_eval_score, n_proj, eta_q16, d_order, d_nd, dist)) != RP_OK) break;
        if ((e = cudaMemcpyAsync(h, d_order, sizeof(int) * M, cudaMemcpyDeviceToHost, c->stream)) != cudaSuccess) break;
        if ((e = cudaMemcpyAsync(h + M, d_nd, sizeof(int), cudaMemcpyDeviceToHost, c->stream)) != cudaSuccess) break;
        if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) break;
        const int nd = h[M];
        if (nd < 1) { st = RP_ERR_STATE; break; }
        int *pick = h + M + 1;
        for (int m = 0; m < P; ++m) pick[m] = h[m % nd];         // the selection order, repeated cyclically
        if ((st = dev_alloc(c, &fin, (size_t)P * dm.N)) != RP_OK) break;
        if ((st = dev_alloc(c, &d_pick, P)) != RP_OK) break;
        if ((e = cudaMemcpyAsync(d_pick, pick, sizeof(int) * P, cudaMemcpyHostToDevice, c->stream)) != cudaSuccess) break;
        k_pick_rows<<<P, 256, 0, c->stream>>>(dm.N, d_pick, out, fin);
        ++g_rp_launches;
        if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) break;      // `pick` is pageable memory
        // the population proper
        c->Ppop = P;
        if ((st = build_population(c)) != RP_OK) break;
        if ((st = install_population(c, fin, nd)) != RP_OK) break;          // rows nd.. repeat the first nd
        if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) break;
        if (n_distinct) *n_distinct = nd;
        if (picked) memcpy(picked, pick, sizeof(int) * P);
    } while (0);
    dev_free(c, lay); dev_free(c, out); dev_free(c, sel); dev_free(c, ok); dev_free(c, prof); dev_free(c, d_order); dev_free(c, d_nd);
    dev_free(c, dist); dev_free(c, fin); dev_free(c, d_pick);
    free(h);
    if (c->Ppop != P) {                      // failed half way: back to a seed population of the right size
        c->Ppop = P;
        const int st2 = build_population(c);
        if (st == RP_OK && e == cudaSuccess) st = st2;
    }
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return st;
}

// Per-level integers of the geometric schedule, from IEEE double operations only.
static void make_schedule(const rp_anneal_params *p, RpLevel *lv)
{
    const double LN2 = 0.6931471805599453094;
    volatile double T = p->t0;
    for (int n = 0; n < p->n_levels; ++n) {
        volatile double Tn = T * p->t_ratio;
        volatile double x = T * LN2;
        x = x * 4294967296.0;
        lv[n].tau = (x >= 1.8e19) ? ~0ull : (u64)floor(x);
        volatile double inv_next = 1.0 / Tn, inv_cur = 1.0 / T;
        volatile double db = inv_next - inv_cur;
        volatile double y = db * (1.0 / LN2);
        y = y * 65536.0;
        lv[n].cq = (y > 0.0) ? ((y >= 1.8e19) ? ~0ull : (u64)floor(y)) : 0ull;
        T = Tn;
    }
}

static int launch_best_check(rp_ctx *c);
static int best_verdict(const rp_ctx *c, const int *sw);

__global__ void k_reset_anneal(i64 *__restrict__ counters, int *__restrict__ status, int *__restrict__ inc_slot,
                               int *__restrict__ done, int *__restrict__ sync, int n_sync)
{
    const int x = threadIdx.x;
    if (x < 8) counters[x] = 0;
    if (x < RP_SW_COUNT) status[x] = 0;
    if (x == 0) { *inc_slot = -1; *done = 0; }
    for (int y = x; y < n_sync; y += blockDim.x) sync[y] = 0;
}

extern "C" int rp_anneal(rp_ctx *c, const rp_anneal_params *p, rp_anneal_stats *stats)
{
    if (!c || !p) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    if (p->n_levels < 1 || p->steps_per_level < 1 || p->n_levels > 100000 || p->steps_per_level > (1 << 22)) return RP_ERR_ARG;
    if (!(p->t0 > 0.0) || !(p->t_ratio > 0.0) || p->t_ratio > 1.0) return RP_ERR_ARG;
    if (!(p->p_reloc >= 0.0) || p->p_reloc > 1.0 || !(p->p_guide >= 0.0) || p->p_guide > 1.0) return RP_ERR_ARG;
    const size_t P = (size_t)c->Ppop;
    const int NL = p->n_levels;
    // schedule
    free(c->h_levels);
    c->h_levels = (RpLevel *)malloc(sizeof(RpLevel) * NL);
    make_schedule(p, c->h_levels);
    const u64 rho_q32 = (u64)floor(p->p_reloc * 4294967296.0);
    const u64 guide_q32 = (u64)floor(p->p_guide * 4294967296.0);
    // accepted-move log
    if (c->log_cap < p->steps_per_level) {
        dev_free(c, c->d_log); c->d_log = nullptr; c->log_cap = 0;
        RP_TRY(dev_alloc(c, &c->d_log, P * (size_t)p->steps_per_level));
        c->log_cap = p->steps_per_level;
    }
    // per-level trace (only when the inspection hook asked for it)
    free_trace(c);
    if (c->trace_on) {
        RP_TRY(dev_alloc(c, &c->d_tr_term, (size_t)NL * P * 3));
        RP_TRY(dev_alloc(c, &c->d_tr_best, (size_t)NL * P * 3));
        RP_TRY(dev_alloc(c, &c->d_tr_inc, (size_t)NL * 3));
        RP_TRY(dev_alloc(c, &c->d_tr_best_step, (size_t)NL * P));
        RP_TRY(dev_alloc(c, &c->d_tr_digest, (size_t)NL * P));
        RP_TRY(dev_alloc(c, &c->d_tr_anc, (size_t)(NL > 1 ? NL - 1 : 1) * P));
        c->trace_levels = NL;
    }
    // counters and status words to zero, incumbent slot to -1 (the incumbent is in d_inc_layout)
    k_reset_anneal<<<1, 256, 0, c->stream>>>(c->d_counters, c->d_status, c->d_inc_slot, c->d_done, c->d_sync, c->Ppop + 1);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());

    cudaEvent_t ev[2] = { nullptr, nullptr };
    if (stats) for (int x = 0; x < 2; ++x) RP_CUDA(cudaEventCreate(&ev[x]));
    float ms_chains = 0.f;
    int st = RP_OK;
    // One launch for all levels where every chain can be resident at once, else one launch per level.
    int all_in_one = 0;
    if (rp_uses_wpc(c->dm) && c->knob_level_launches != 1) st = rp_upload_levels(c, NL);
    if (stats) cudaEventRecord(ev[0], c->stream);
    if (st == RP_OK) st = rp_launch_anneal_all(c, NL, p, rho_q32, guide_q32, &all_in_one);
    if (all_in_one) c->cur = (c->cur + NL) & 1;       // the kernel has left both ancestor tables and both cell tables current
    for (int n = 0; n < NL && st == RP_OK && !all_in_one; ++n) {
        st = rp_launch_anneal_level(c, n, NL, p, rho_q32, guide_q32);
        c->cur = 1 - c->cur;          // the terminal states are the next level's sources
        { int *sw = c->d_anc; c->d_anc = c->d_anc_next; c->d_anc_next = sw; }
        { int *sw = c->d_wloc; c->d_wloc = c->d_wloc_next; c->d_wloc_next = sw; }
    }
    if (stats) cudaEventRecord(ev[1], c->stream);
    // Validate(x*) and the full rescoring of the incumbent follow in the same stream, so that
    // rp_best finds them done
    c->best_ready = 0;
    if (st == RP_OK) st = launch_best_check(c);
    // one synchronisation: the counters and the status words ride back in the pinned block
    i64 *cn = c->h_pin;                       // [8] counters
    int *sw = (int *)(c->h_pin + 56);         // status words
    cudaError_t e = cudaMemcpyAsync(cn, c->d_counters, sizeof(i64) * 8, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(sw, c->d_status, sizeof(int) * RP_SW_COUNT, cudaMemcpyDeviceToHost, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (stats) {
        if (e == cudaSuccess) cudaEventElapsedTime(&ms_chains, ev[0], ev[1]);
        for (int x = 0; x < 2; ++x) cudaEventDestroy(ev[x]);
    }
    if (st == RP_OK && e != cudaSuccess) { g_rp_last_cuda_error = (int)e; st = RP_ERR_CUDA; }
    RP_TRY(st);
    if (sw[RP_SW_POOL]) { c->stage = 2; c->best_ready = 0; return RP_ERR_STATE; }     // slice pool exhausted: an internal invariant broke
    if (sw[RP_SW_TIMEOUT]) {
        // A bounded device-side wait ran out: that level's barrier and every later level were
        // skipped, so the population is not a population any more.  Back to "placed": only
        // rp_pack_rows (which rebuilds it from the seed) and rp_destroy make sense now.
        c->stage = 2;
        c->best_ready = 0;
        return RP_ERR_TIMEOUT;
    }
    if (stats) {
        stats->proposed = cn[0]; stats->feasible = cn[1]; stats->accepted = cn[2]; stats->improved = cn[3];
        stats->move_bytes = cn[4]; stats->gather_bytes = cn[5]; stats->staging_bytes = cn[6];
        stats->kernel_launches = all_in_one ? 1 : (int64_t)NL * ((rp_uses_slices(c->dm) ? 3 : 1) + (rp_uses_warp_chains(c) ? 1 : 0));
        stats->ms_chains = ms_chains;
    }
    c->best_verdict = best_verdict(c, sw);
    c->best_ready = 1;
    c->stage = 4;
    return RP_OK;
}

// Validate(x*) on the device: coverage / capacity / non-empty cells, and a full rescoring of the
// incumbent; the three score tuples the verdict needs are queued into the pinned block.
static int launch_best_check(rp_ctx *c)
{
    stage_mark(c, RP_EV_BEST_0, c->stream);
    RP_TRY(rp_launch_validate(c));
    RP_TRY(ensure_eval_scratch(c, 1, false));
    RP_TRY(rp_launch_cells_from_layouts(c, c->d_inc_layout, 1, c->d_eval_cells));
    RP_TRY(rp_launch_eval(c, c->d_eval_cells, 1, nullptr, nullptr, c->d_best_score, c->d_best_f64));
    stage_mark(c, RP_EV_BEST_1, c->stream);
    RP_CUDA(cudaMemcpyAsync(c->h_pin + 16, c->d_inc_score, sizeof(i64) * 3, cudaMemcpyDeviceToHost, c->stream));
    RP_CUDA(cudaMemcpyAsync(c->h_pin + 19, c->d_best_score, sizeof(i64) * 3, cudaMemcpyDeviceToHost, c->stream));
    RP_CUDA(cudaMemcpyAsync(c->h_pin + 22, c->d_seed_score, sizeof(i64) * 3, cudaMemcpyDeviceToHost, c->stream));
    return RP_OK;
}

// After the stream has been synchronised: the verdict from the pinned block and the status words.
static int best_verdict(const rp_ctx *c, const int *sw)
{
    const i64 *inc = c->h_pin + 16, *full = c->h_pin + 19, *seed = c->h_pin + 22;
    bool ok = !sw[RP_SW_VALIDATE] && !sw[RP_SW_BAD_LAYOUT];
    ok = ok && inc[0] == full[0] && inc[1] == full[1] && inc[2] == full[2];
    // non-regression: not worse than the best member of the initial population
    const bool worse = (seed[0] != inc[0]) ? (seed[0] < inc[0]) : (seed[1] != inc[1]) ? (seed[1] < inc[1]) : (seed[2] < inc[2]);
    ok = ok && !worse;
    return ok ? RP_OK : RP_ERR_INVALID_PLAN;
}

extern "C" int rp_best(rp_ctx *c, int32_t *cell_of_sample, int64_t *score_fx, double *score_f64)
{
    if (!c) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    const RpDims &dm = c->dm;
    int *sw = (int *)(c->h_pin + 56);
    const bool fresh = !c->best_ready;          // rp_anneal validates its incumbent before it returns
    if (fresh) {
        RP_TRY(reset_status(c));
        RP_TRY(launch_best_check(c));
        RP_CUDA(cudaMemcpyAsync(sw, c->d_status, sizeof(int) * RP_SW_COUNT, cudaMemcpyDeviceToHost, c->stream));
    }
    RP_TRY(copy_out(c, cell_of_sample, c->d_inc_layout, sizeof(int) * (size_t)dm.N));
    RP_TRY(copy_out(c, score_fx, c->d_inc_score, sizeof(i64) * 3));
    RP_TRY(copy_out(c, score_f64, c->d_best_f64, sizeof(double) * 3));
    // Outputs are complete when the call returns.
    if (fresh || cell_of_sample || score_fx || score_f64) RP_CUDA(cudaStreamSynchronize(c->stream));
    if (fresh) { c->best_verdict = best_verdict(c, sw); c->best_ready = 1; }
    return c->best_verdict;
}

// ---------------------------------------------------------------------------------------
// inspection hooks
// ---------------------------------------------------------------------------------------
__global__ void k_cell_stats(const unsigned short *__restrict__ cells, const int *__restrict__ t, int N, int K,
                             i64 *__restrict__ T, i64 *__restrict__ Q, int *__restrict__ cnt)
{
    for (int c = threadIdx.x; c < K; c += blockDim.x) { T[c] = 0; Q[c] = 0; cnt[c] = 0; }
    __syncthreads();
    for (int i = threadIdx.x; i < N; i += blockDim.x) {
        int c = cells[i];
        atomicAdd((u64 *)&T[c], (u64)t[i]);
        atomicAdd((u64 *)&Q[c], (u64)t[i] * (u64)t[i]);
        atomicAdd(&cnt[c], 1);
    }
}

extern "C" int rp_debug_set_stage_timing(int on) { g_stage_timing = on ? 1 : 0; return RP_OK; }

extern "C" int rp_debug_stage_times(rp_ctx *c, double *ms)
{
    if (!c || !ms) return RP_ERR_ARG;
    if (!c->ev_stage[0]) return RP_ERR_STATE;
    RP_CUDA(cudaStreamSynchronize(c->stream));
    static const int pairs[6][2] = { { RP_EV_K1_0, RP_EV_K1_1 }, { RP_EV_K2_0, RP_EV_K2_1 }, { RP_EV_K2_1, RP_EV_K3_1 },
                                     { RP_EV_PACK_0, RP_EV_PACK_1 }, { RP_EV_SEED_0, RP_EV_SEED_1 }, { RP_EV_BEST_0, RP_EV_BEST_1 } };
    for (int x = 0; x < 6; ++x) {
        ms[x] = -1.0;
        const unsigned need = (1u << pairs[x][0]) | (1u << pairs[x][1]);
        if ((c->ev_recorded & need) != need) continue;
        float t = 0.f;
        if (cudaEventSynchronize(c->ev_stage[pairs[x][1]]) == cudaSuccess &&
            cudaEventElapsedTime(&t, c->ev_stage[pairs[x][0]], c->ev_stage[pairs[x][1]]) == cudaSuccess) ms[x] = t;
        else cudaGetLastError();
    }
    return RP_OK;
}

extern "C" int rp_debug_set_knob(rp_ctx *c, int knob, int64_t value)
{
    if (!c || value < 0) return RP_ERR_ARG;
    switch (knob) {
        case RP_KNOB_BARRIER_WORKSPACE:
            if (value > (1 << 20) || (value & 15) || (value && value < 64)) return RP_ERR_ARG;
            c->knob_le_ws_cap = (int)value; return RP_OK;
        case RP_KNOB_WAIT_POLLS:
            if (value > (1 << 22)) return RP_ERR_ARG;
            c->knob_wait_polls = (int)value; return RP_OK;
        case RP_KNOB_STALL_ONE_CHAIN:
            c->knob_stall = value ? 1 : 0; return RP_OK;
        case RP_KNOB_LAUNCH_PER_LEVEL:
            if (value > 2) return RP_ERR_ARG;
            c->knob_level_launches = (int)value; return RP_OK;
        case RP_KNOB_RANK_LOAD_SLICES:
            if (value > 2) return RP_ERR_ARG;
            c->knob_slices = (int)value; return RP_OK;
        case RP_KNOB_CHAIN_KERNEL:
            if (value > 2) return RP_ERR_ARG;
            c->knob_chain_kernel = (int)value; return RP_OK;
        default: return RP_ERR_ARG;
    }
}

__global__ void k_gather_slices(const int *__restrict__ W, const int *__restrict__ tab, int LP, int *__restrict__ out)
{
    const int rg = blockIdx.x;
    const int *src = W + (size_t)tab[rg] * LP;
    for (int x = threadIdx.x; x < LP; x += blockDim.x) out[(size_t)rg * LP + x] = src[x];
}

extern "C" int rp_debug_set_trace(rp_ctx *c, int on)
{
    if (!c) return RP_ERR_ARG;
    c->trace_on = on ? 1 : 0;
    return RP_OK;
}

extern "C" int rp_debug_dump(rp_ctx *c, int what, int32_t index, void *buf, int64_t bytes)
{
    if (!c || !buf) return RP_ERR_ARG;
    const RpDims &dm = c->dm;
    const size_t P = (size_t)c->Ppop;
    const void *src = nullptr;
    size_t need = 0;
    void *tmp = nullptr;
    int st = RP_OK;
    int member = -1;
    if (what >= RP_DUMP_POPULATION && what <= RP_DUMP_ESUM) {
        if (c->stage < 3) return RP_ERR_STATE;
        if (what != RP_DUMP_POPULATION) {
            if (index < 0 || index >= c->Ppop) return RP_ERR_ARG;
            RP_CUDA(cudaMemcpyAsync(&member, c->d_anc + index, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
            RP_CUDA(cudaStreamSynchronize(c->stream));
        }
    }
    switch (what) {
        case RP_DUMP_LAGG: if (c->stage < 1) return RP_ERR_STATE; src = c->d_Lagg; need = sizeof(i64) * dm.L * dm.E; break;
        case RP_DUMP_Q: if (c->stage < 2) return RP_ERR_STATE; src = c->d_q; need = sizeof(int) * (size_t)dm.N * dm.LP; break;
        case RP_DUMP_SEED_LAYOUT: if (c->stage < 3) return RP_ERR_STATE; src = c->d_seed_layout; need = sizeof(int) * dm.N; break;
        case RP_DUMP_POPULATION: {
            need = sizeof(int) * P * dm.N;
            if ((st = dev_alloc(c, (int **)&tmp, P * dm.N)) != RP_OK) return st;
            k_gather_cells<<<c->Ppop, 256, 0, c->stream>>>(c->buf[c->cur].blob, c->bl, c->d_anc, dm.N, nullptr, (int *)tmp);
            ++g_rp_launches;
            src = tmp;
            break;
        }
        case RP_DUMP_W:
            if (rp_uses_slices(dm)) {          // the member's slices, gathered through its table
                need = sizeof(int) * (size_t)dm.RG * dm.LP;
                if ((st = dev_alloc(c, (int **)&tmp, (size_t)dm.RG * dm.LP)) != RP_OK) return st;
                k_gather_slices<<<dm.RG, 128, 0, c->stream>>>(c->d_W, (const int *)(c->buf[c->cur].blob + (size_t)member * c->bl.bytes + c->bl.off_wtab),
                                                              dm.LP, (int *)tmp);
                ++g_rp_launches;
                src = tmp;
                break;
            }
            {
            int cell = 0;
            RP_CUDA(cudaMemcpyAsync(&cell, c->d_wloc + member, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
            RP_CUDA(cudaStreamSynchronize(c->stream));
            src = c->d_W + (size_t)cell * dm.RG * dm.LP; need = sizeof(int) * (size_t)dm.RG * dm.LP; break;
            }
        case RP_DUMP_ESUM: src = c->buf[c->cur].blob + (size_t)member * c->bl.bytes + c->bl.off_Esum; need = sizeof(i64) * dm.RG; break;
        case RP_DUMP_CELL_T: case RP_DUMP_CELL_Q: case RP_DUMP_CELL_CNT: {
            size_t K = dm.K;
            if ((st = dev_alloc(c, (i64 **)&tmp, 3 * K)) != RP_OK) return st;
            i64 *T = (i64 *)tmp, *Q = T + K;
            int *cnt = (int *)(Q + K);
            k_cell_stats<<<1, 256, 0, c->stream>>>((const unsigned short *)(c->buf[c->cur].blob + (size_t)member * c->bl.bytes + c->bl.off_cell),
                                                   c->d_t, dm.N, dm.K, T, Q, cnt);
            ++g_rp_launches;
            if (what == RP_DUMP_CELL_T) { src = T; need = sizeof(i64) * K; }
            else if (what == RP_DUMP_CELL_Q) { src = Q; need = sizeof(i64) * K; }
            else { src = cnt; need = sizeof(int) * K; }
            break;
        }
        case RP_DUMP_TRACE_TERM: src = c->d_tr_term; need = sizeof(i64) * 3 * P * c->trace_levels; break;
        case RP_DUMP_TRACE_BEST: src = c->d_tr_best; need = sizeof(i64) * 3 * P * c->trace_levels; break;
        case RP_DUMP_TRACE_BEST_STEP: src = c->d_tr_best_step; need = sizeof(int) * P * c->trace_levels; break;
        case RP_DUMP_TRACE_DIGEST: src = c->d_tr_digest; need = sizeof(u64) * P * c->trace_levels; break;
        case RP_DUMP_TRACE_ANC: src = c->d_tr_anc; need = sizeof(int) * P * (c->trace_levels > 1 ? c->trace_levels - 1 : 0); break;
        case RP_DUMP_TRACE_INCUMBENT: src = c->d_tr_inc; need = sizeof(i64) * 3 * c->trace_levels; break;
        case RP_DUMP_EVAL_W:
            if (index < 0 || index >= c->eval_W_n) return RP_ERR_ARG;
            src = c->d_eval_W + (size_t)index * dm.RG * dm.LP; need = sizeof(int) * (size_t)dm.RG * dm.LP; break;
        case RP_DUMP_SELECT_DIST:
            if (!c->d_sel_dist) return RP_ERR_STATE;
            src = c->d_sel_dist; need = sizeof(i64) * P * P; break;
        default: return RP_ERR_ARG;
    }
    if (what >= RP_DUMP_TRACE_TERM && what <= RP_DUMP_TRACE_INCUMBENT && c->trace_levels == 0) { dev_free(c, tmp); return RP_ERR_STATE; }
    if ((int64_t)need != bytes) { dev_free(c, tmp); return RP_ERR_ARG; }
    cudaError_t e = cudaSuccess;
    if (need) e = cudaMemcpyAsync(buf, src, need, cudaMemcpyDefault, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    dev_free(c, tmp);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return RP_OK;
}

__global__ void k_dbg_nl2(const u32 *x, u64 *out, long long n)
{
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = rp_nl2(x[i]);
}
__global__ void k_dbg_exp2neg(const u64 *z, u64 *out, long long n)
{
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = rp_exp2neg(z[i]);
}
__global__ void k_dbg_philox(const u32 *ctr, u32 k0, u32 k1, u32 *out, long long n)
{
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        uint4 r = rp_philox(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3], k0, k1);
        out[4 * i] = r.x; out[4 * i + 1] = r.y; out[4 * i + 2] = r.z; out[4 * i + 3] = r.w;
    }
}

// Read bandwidth of a buffer that stays in L2: every thread sums 16-byte pieces of it, the whole
// buffer `reps` times over; the figure is the denominator for kernels whose operands L2 serves.
__global__ void k_dbg_l2_read(const int4 *__restrict__ buf, long long n4, int reps, int *__restrict__ sink)
{
    int acc = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (int r = 0; r < reps; ++r)
        for (long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x; x < n4; x += stride) {
            const int4 v = __ldcg(buf + x);
            acc += v.x ^ v.y ^ v.z ^ v.w;
        }
    if (acc == 0x7fffffff) *sink = acc;          // never true for the zeroed buffer: keeps the loads alive
}

extern "C" int rp_debug_chain_kernel(rp_ctx *c, int32_t *which)
{
    if (!c || !which) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    *which = rp_uses_warp_chains(c) ? 2 : (rp_uses_wpc(c->dm) ? 0 : 1);
    return RP_OK;
}

extern "C" int rp_debug_l2_read_rate(int64_t bytes, int32_t reps, double *gb_per_s)
{
    if (!gb_per_s || bytes < (1 << 20) || bytes > (1ll << 31) || reps < 1 || reps > 10000) return RP_ERR_ARG;
    int4 *buf = nullptr;
    int *sink = nullptr;
    RP_CUDA(cudaMalloc((void **)&buf, (size_t)bytes));
    if (cudaMalloc((void **)&sink, sizeof(int)) != cudaSuccess) { cudaFree(buf); return RP_ERR_CUDA; }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaMemset(buf, 0, (size_t)bytes);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        const long long n4 = bytes / 16;
        k_dbg_l2_read<<<148 * 8, 256>>>(buf, n4, 2, sink);              // warm the cache
        cudaEventRecord(e0);
        k_dbg_l2_read<<<148 * 8, 256>>>(buf, n4, reps, sink);
        cudaEventRecord(e1);
        g_rp_launches += 2;
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(buf); cudaFree(sink);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    *gb_per_s = (double)bytes * reps / (ms * 1e-3) / 1e9;
    return RP_OK;
}

template <class TI, class TO, class F>
static int dbg_map(const TI *in, size_t in_per, TO *out, size_t out_per, int64_t n, F launch)
{
    if (!in || !out || n < 0) return RP_ERR_ARG;
    if (n == 0) return RP_OK;
    TI *din = nullptr; TO *dout = nullptr;
    RP_CUDA(cudaMalloc((void **)&din, sizeof(TI) * (size_t)n * in_per));
    if (cudaMalloc((void **)&dout, sizeof(TO) * (size_t)n * out_per) != cudaSuccess) { cudaFree(din); return RP_ERR_CUDA; }
    cudaError_t e = cudaMemcpy(din, in, sizeof(TI) * n * in_per, cudaMemcpyDefault);
    if (e == cudaSuccess) { launch(din, dout); ++g_rp_launches; e = cudaGetLastError(); }
    if (e == cudaSuccess) e = cudaMemcpy(out, dout, sizeof(TO) * n * out_per, cudaMemcpyDefault);
    cudaFree(din); cudaFree(dout);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return RP_OK;
}

extern "C" int rp_debug_nl2(const uint32_t *x, uint64_t *out, int64_t n)
{
    return dbg_map<u32, u64>(x, 1, (u64 *)out, 1, n, [&](u32 *a, u64 *b) { k_dbg_nl2<<<(unsigned)((n + 255) / 256), 256>>>(a, b, n); });
}
extern "C" int rp_debug_exp2neg(const uint64_t *z, uint64_t *out, int64_t n)
{
    return dbg_map<u64, u64>((const u64 *)z, 1, (u64 *)out, 1, n, [&](u64 *a, u64 *b) { k_dbg_exp2neg<<<(unsigned)((n + 255) / 256), 256>>>(a, b, n); });
}
extern "C" int rp_debug_philox(const uint32_t *ctr, const uint32_t key[2], uint32_t *out, int64_t n)
{
    if (!key) return RP_ERR_ARG;
    const u32 k0 = key[0], k1 = key[1];
    return dbg_map<u32, u32>(ctr, 4, out, 4, n, [&](u32 *a, u32 *b) { k_dbg_philox<<<(unsigned)((n + 255) / 256), 256>>>(a, k0, k1, b, n); });
}
