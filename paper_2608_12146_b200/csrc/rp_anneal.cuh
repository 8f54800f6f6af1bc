// Shared pieces of the two chain kernels of the population annealing (Algorithm 3):
// kernel arguments, the state-independent step record, the proposal rule and the
// vectorised two-slice scoring pass.
#pragma once
#include "rp_score.cuh"

// Outputs of the level barrier (incumbent, next ancestors, per-level trace).
struct LevelOut {
    int *done;                 // arrival counter of the chain CTAs (zero between launches)
    int *anc_out;              // [P_pop] ancestors for the next level
    int *wloc_out;             // [P_pop] W cells for the next level
    int *scratch;              // [6*P_pop] ints
    u64 *F;                    // [P_pop] cumulative resampling weights
    int *inc_layout;           // [N]
    i64 *inc_score;            // [3]
    // Chains that keep a snapshot of their trajectory-best layout (null otherwise: the barrier then
    // rebuilds the winner's layout from its move log).  A chain writes its row only when it
    // strictly beats the incumbent, and then the barrier of that level names a new incumbent
    // among the writers: the row of the current incumbent's slot is never overwritten unnoticed.
    unsigned short *cand_layout;   // [P_pop][N]
    int *inc_slot;                 // slot whose row holds the incumbent, -1 = inc_layout is current
    int *anc_cur;                  // the ancestor table the call started from (one launch for all levels: both are set at the end)
    i64 *tr_term, *tr_best, *tr_inc;     // trace (nullable)
    int *tr_best_step, *tr_anc;
    u64 *tr_digest;
};

struct RpLevelDev { u64 tau, cq; u32 resample_x, pad; };   // per-level schedule integers on the device

struct AnnealArgs {
    RpDims dm;
    RpBlob bl;
    RpStatic sl;
    const int *t, *q;
    const char *static_blk;
    const char *blob_src;  char *blob_dst;
    int *W;                          // rank-load cells [2*P_pop][RG][LP]
    const int *wloc_src;             // [P_pop] cell of each member's W at the start of the level
    int *wloc_dst;                   // [P_pop] cell each slot works in; rewritten by the level barrier for the next level
    const int *anc;
    int level, steps, log_cap, Ppop, last;
    int w_on_chip;                   // W is staged in shared memory: every level moves it anyway
    // Slice mode (rank loads too large for one cell copy per replaced member): W is a pool of
    // 2*P_pop*RG slices of L*P ints, a member's blob carries the slice of each of its row-shards,
    // and a child shares its ancestor's slices until it rewrites them (an accepted move rewrites
    // whole slices anyway, so leaving a shared slice costs no copy).
    int slices;
    const int *wref;                 // [2*P_pop*RG] holders of each slice at the start of the level
    const int *wfree;                // free slices in ascending order; member j's spares are entries j*RG .. j*RG+RG-1
    const int *wfree_head;           // [1] entries in the list
    unsigned smem_bytes;             // dynamic shared memory of the launch
    u64 tau, cq, rho_q32, guide_q32;
    u32 key0, key1;
    u32 resample_x;                  // Philox(0, level, 0, 3).x, the word behind the resampling offset (computed on the host)
    // One launch for all levels (every chain resident at once): the levels' schedule, the two blob
    // buffers by name, which of them the call starts from, the arrival counter and the time a chain
    // may wait for the others.
    int n_levels, cur0;
    const RpLevelDev *levels;
    char *blob_b0, *blob_b1;
    int *sync;
    u64 bar_timeout_ns;
    int wait_polls;                  // limit of every bounded wait on a bulk-copy barrier (polls)
    int stall_test;                  // inspection hook: after its loads have landed, chain 0 waits once more on a
                                     // barrier phase that nothing completes, so that the wait runs out
    unsigned le_ws_cap;              // inspection hook: shared-memory bytes the level barrier may use (0 = all)
    i64 *term, *best;
    int *best_step, *best_nlog;
    u64 *digest;
    uint2 *log;
    i64 *counters;
    int *status;
    LevelOut lo;
};

#define SPEC 32                 // steps speculated per round = lanes of the leading warp

struct StepRec {                // everything about a step that does not depend on the chain state
    u32 flags;                  // bit0 relocation, bit1 guided, bit2 accept threshold saturated
    int i0, i1, i2, i3;         // candidate indices (samples, or cells for relocation targets)
    u32 bz;                     // word of the attention-key coin
    u64 thr;                    // (tau * -log2(u)) >> 32, Q32
};
struct MoveS { int reloc, i, i2, c1, c2; };

// Random words of step k of chain slot j at this level -> the step record.
// Purposes: 0 = proposal words A, 1 = proposal words B, 2 = accept word.
// The uniform branch is stored as a tournament between a candidate and itself, so that the
// proposal rule below needs no branch on it.
__device__ __forceinline__ StepRec rp_make_step_rec(const AnnealArgs &A, int level, u64 tau, u32 k, u32 j)
{
    const RpDims &dm = A.dm;
    const uint4 a = rp_philox(k, (u32)level, j, 0u, A.key0, A.key1);
    const uint4 b = rp_philox(k, (u32)level, j, 1u, A.key0, A.key1);
    const uint4 xw = rp_philox(k, (u32)level, j, 2u, A.key0, A.key1);
    const bool reloc = (u64)a.x < A.rho_q32, guided = (u64)a.y < A.guide_q32;
    StepRec r;
    r.i0 = rp_pick(a.z, dm.N);
    if (!guided) {
        r.i1 = r.i0;
        r.i2 = reloc ? rp_pick(a.w, dm.K) : rp_pick(a.w, dm.N);
        r.i3 = r.i2;
    } else {
        r.i1 = rp_pick(a.w, dm.N);
        r.i2 = reloc ? rp_pick(b.x, dm.K) : rp_pick(b.x, dm.N);
        r.i3 = reloc ? rp_pick(b.y, dm.K) : rp_pick(b.y, dm.N);
    }
    r.bz = b.z;
    const u64 nl = rp_nl2(xw.x);
    const u64 hi = __umul64hi(tau, nl), lo = tau * nl;
    const bool sat = (hi >> 30) != 0;
    r.thr = (hi << 32) | (lo >> 32);
    r.flags = (reloc ? 1u : 0u) | (guided ? 2u : 0u) | (sat ? 4u : 0u);
    return r;
}

// Tables of the chain state the proposal rule reads (all in shared memory).  The three
// per-cell arrays are caches kept in step with the state: the attention cost of the cell,
// and the cost J and the attention part A of the row-shard the cell belongs to.
struct RpChainView {
    const unsigned short *cell_of;
    const int *T, *cnt, *tt;
    const i64 *attkey, *Jcell, *Acell;
};

// GuidedProposal + feasibility of one step against the current state.
//   Tournament of two.  Source candidates i0, i1; the comparison key is the attention cost
//   of the candidate's cell with probability Afx/Jfx of the first candidate's row-shard
//   (bz * Jfx < Afx * 2^32), else the row-shard cost Jfx; source = larger key (tie: first).
//   Target candidates i2, i3 (samples for a swap, cells for a relocation); target = smaller
//   key (tie: first).  The uniform branch arrives as i1 == i0 and i3 == i2.
// Feasible = distinct cells, both cells within the token cap afterwards, no cell emptied.
__device__ __forceinline__ bool rp_propose(const RpDims &dm, const RpChainView &v, const StepRec &r, MoveS &m)
{
    const bool reloc = r.flags & 1u;
    const int ca = v.cell_of[r.i0], cb = v.cell_of[r.i1];
    const int xa = reloc ? r.i2 : (int)v.cell_of[r.i2];
    const int xb = reloc ? r.i3 : (int)v.cell_of[r.i3];
    const u64 Ja = (u64)v.Jcell[ca], Aa = (u64)v.Acell[ca];
    const u64 lh = __umul64hi((u64)r.bz, Ja), ll = (u64)r.bz * Ja;
    const u64 rh = Aa >> 32, rl = Aa << 32;
    const bool use_att = (lh < rh) || (lh == rh && ll < rl);
    const i64 *key = use_att ? v.attkey : v.Jcell;
    const i64 ka = key[ca], kb = key[cb], ta = key[xa], tb = key[xb];
    const bool src_b = kb > ka, dst_b = tb < ta;
    m.reloc = reloc;
    m.i = src_b ? r.i1 : r.i0;
    m.c1 = src_b ? cb : ca;
    m.c2 = dst_b ? xb : xa;
    m.i2 = reloc ? -1 : (dst_b ? r.i3 : r.i2);
    if (m.c1 == m.c2) return false;
    const int ti = v.tt[m.i];
    if (reloc) return (v.cnt[m.c1] > 1) && (v.T[m.c2] + ti <= dm.C);
    const int t2 = v.tt[m.i2];
    return (v.T[m.c1] - ti + t2 <= dm.C) && (v.T[m.c2] - t2 + ti <= dm.C);
}

// The same rule, also handing back the lengths of the moved samples (the decision needs them again,
// and for long windows they come from global memory).
__device__ __forceinline__ bool rp_propose_len(const RpDims &dm, const RpChainView &v, const StepRec &r, MoveS &m, int &ti_out, int &t2_out)
{
    const bool reloc = r.flags & 1u;
    const int ca = v.cell_of[r.i0], cb = v.cell_of[r.i1];
    const int xa = reloc ? r.i2 : (int)v.cell_of[r.i2];
    const int xb = reloc ? r.i3 : (int)v.cell_of[r.i3];
    const u64 Ja = (u64)v.Jcell[ca], Aa = (u64)v.Acell[ca];
    const u64 lh = __umul64hi((u64)r.bz, Ja), ll = (u64)r.bz * Ja;
    const u64 rh = Aa >> 32, rl = Aa << 32;
    const bool use_att = (lh < rh) || (lh == rh && ll < rl);
    const i64 *key = use_att ? v.attkey : v.Jcell;
    const i64 ka = key[ca], kb = key[cb], ta = key[xa], tb = key[xb];
    const bool src_b = kb > ka, dst_b = tb < ta;
    m.reloc = reloc;
    m.i = src_b ? r.i1 : r.i0;
    m.c1 = src_b ? cb : ca;
    m.c2 = dst_b ? xb : xa;
    m.i2 = reloc ? -1 : (dst_b ? r.i3 : r.i2);
    if (m.c1 == m.c2) return false;
    const int ti = v.tt[m.i];
    ti_out = ti; t2_out = 0;
    if (reloc) return (v.cnt[m.c1] > 1) && (v.T[m.c2] + ti <= dm.C);
    const int t2 = v.tt[m.i2];
    t2_out = t2;
    return (v.T[m.c1] - ti + t2 <= dm.C) && (v.T[m.c2] - t2 + ti <= dm.C);
}

__device__ __forceinline__ int max4(const int4 &v) { return max(max(v.x, v.y), max(v.z, v.w)); }

// Tentative rank loads of the two touched row-shards, W1' = W1 - d and W2' = W2 + d with
// d = q[i] - q[i2] (relocation: d = q[i]), in two halves: all loads of a pass are issued before any is consumed.  NTH threads cooperate (tid in
// [0,NTH)); whole warps must call.  16-byte loads, CH chunks per thread in flight per pass;
// ranks of a layer are reduced by segmented shuffles; needs P a power of two, 4 <= P <= 128.
template <int CH>
struct RpSliceRegs { int4 d[CH], a[CH], b[CH]; };

template <int CH, int NTH>
__device__ __forceinline__ void rp_slices_load(RpSliceRegs<CH> &r, int base, int nchunks, const int4 *__restrict__ qi,
                                               const int4 *__restrict__ q2, const int4 *w1, const int4 *w2, int tid)
{
#pragma unroll
    for (int u = 0; u < CH; ++u) {
        const int c = base + u * NTH + tid;
        if (c < nchunks) {
            r.d[u] = __ldg(qi + c);
            if (q2) { const int4 o = __ldg(q2 + c); r.d[u].x -= o.x; r.d[u].y -= o.y; r.d[u].z -= o.z; r.d[u].w -= o.w; }
            r.a[u] = w1[c];
            r.b[u] = w2[c];
        }
    }
}

template <int CH, int NTH>
__device__ __forceinline__ void rp_slices_reduce(const RpSliceRegs<CH> &r, int base, int nchunks, int lanes_per_layer,
                                                 int4 *s1, int4 *s2, int tid, i64 &e1, i64 &e2)
{
    const int lane = tid & 31;
#pragma unroll
    for (int u = 0; u < CH; ++u) {
        const int c = base + u * NTH + tid;
        int m1 = 0, m2 = 0;
        if (c < nchunks) {
            const int4 v1 = make_int4(r.a[u].x - r.d[u].x, r.a[u].y - r.d[u].y, r.a[u].z - r.d[u].z, r.a[u].w - r.d[u].w);
            const int4 v2 = make_int4(r.b[u].x + r.d[u].x, r.b[u].y + r.d[u].y, r.b[u].z + r.d[u].z, r.b[u].w + r.d[u].w);
            s1[c] = v1;
            s2[c] = v2;
            m1 = max4(v1);
            m2 = max4(v2);
        }
        for (int o = lanes_per_layer >> 1; o; o >>= 1) {
            m1 = max(m1, __shfl_xor_sync(0xffffffffu, m1, o));
            m2 = max(m2, __shfl_xor_sync(0xffffffffu, m2, o));
        }
        if ((lane & (lanes_per_layer - 1)) == 0 && c < nchunks) { e1 += m1; e2 += m2; }
    }
}

__device__ __forceinline__ i64 warp_max_i64(i64 v)
{
    for (int o = 16; o; o >>= 1) { i64 x = __shfl_xor_sync(0xffffffffu, v, o); v = x > v ? x : v; }
    return v;
}
// Warp maximum of non-negative 64-bit values with two reduction instructions: the largest high
// word, then the largest low word among the lanes that hold it.
__device__ __forceinline__ i64 warp_max_nonneg_i64(i64 v)
{
    const u32 hi = (u32)((u64)v >> 32), lo = (u32)v;
    const u32 mh = __reduce_max_sync(0xffffffffu, hi);
    const u32 ml = __reduce_max_sync(0xffffffffu, hi == mh ? lo : 0u);
    return (i64)(((u64)mh << 32) | ml);
}
__device__ __forceinline__ i64 warp_sum_i64(i64 v)
{
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- bulk asynchronous copies (TMA, untiled) and their mbarrier -----------------------------
// Both addresses and the size must be multiples of 16 bytes.
__device__ __forceinline__ u32 rp_smem_addr(const void *p) { return (u32)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void rp_mbar_init(u64 *mbar, u32 count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(rp_smem_addr(mbar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void rp_mbar_expect_tx(u64 *mbar, u32 bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(rp_smem_addr(mbar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void rp_bulk_g2s(void *smem_dst, const void *gmem_src, u32 bytes, u64 *mbar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(rp_smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(rp_smem_addr(mbar)) : "memory");
}
// Bounded wait on a barrier phase; false when the limit ran out.
__device__ __forceinline__ bool rp_mbar_wait(u64 *mbar, u32 parity, int limit)
{
    const u32 addr = rp_smem_addr(mbar);
    for (int it = 0; it < limit; ++it) {
        u32 done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void rp_bulk_s2g(void *gmem_dst, const void *smem_src, u32 bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gmem_dst), "r"(rp_smem_addr(smem_src)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void rp_bulk_commit_wait()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void rp_fence_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---- chain state in and out of shared memory ---------------------------------------------
// Shared-memory front of both chain kernels: [blob][static tables][W when it lives on chip].
// The blob of the ancestor, the static block and (on chip) the ancestor's W arrive by bulk
// copies on one mbarrier; W kept in global memory is copied by all threads.
// Cell that holds the rank loads of ancestor `src` when this level starts.  With W on chip every
// member works in its own cell m or P + m and all members sit in the same half, so the half of
// this slot's own entry tells where the ancestor's is: no load that depends on `src`.
__device__ __forceinline__ int rp_src_cell(const AnnealArgs &A, int src, int j)
{
    if (A.w_on_chip) return (A.wloc_src[j] >= A.Ppop) ? A.Ppop + src : src;
    return A.wloc_src[src];
}

template <int NT, bool WS>
__device__ __forceinline__ bool rp_chain_load(const AnnealArgs &A, int src, int j, char *sm_blob, char *sm_static,
                                              int *Wsm, u64 *mbar, int tid, int src_cell, int dst_cell)
{
    const RpDims &dm = A.dm;
    const size_t wn = (size_t)dm.RG * dm.LP;
    const int *ws = A.W + (size_t)src_cell * wn;
    const bool w_bulk = WS && ((wn & 3) == 0);
    if (tid == 0) {
        rp_mbar_init(mbar, 1);
        const u32 total = (u32)A.bl.bytes + (u32)A.sl.bytes + (w_bulk ? (u32)(wn * 4) : 0u);
        rp_mbar_expect_tx(mbar, total);
        rp_bulk_g2s(sm_blob, A.blob_src + (size_t)src * A.bl.bytes, (u32)A.bl.bytes, mbar);
        rp_bulk_g2s(sm_static, A.static_blk, (u32)A.sl.bytes, mbar);
        if (w_bulk)
            for (size_t off = 0; off < wn * 4; off += 32768) {
                const u32 n = (u32)((wn * 4 - off) < 32768 ? (wn * 4 - off) : 32768);
                rp_bulk_g2s((char *)Wsm + off, (const char *)ws + off, n, mbar);
            }
    }
    if (!w_bulk && !A.slices && (WS || src_cell != dst_cell)) {      // a sole child works on in its ancestor's cell
        int *wd = WS ? Wsm : A.W + (size_t)dst_cell * wn;
        if ((wn & 3) == 0) {
            const int4 *ws4 = (const int4 *)ws;
            int4 *wd4 = (int4 *)wd;
#pragma unroll 8
            for (size_t x = tid; x < wn / 4; x += NT) wd4[x] = __ldg(ws4 + x);
        } else {
            for (size_t x = tid; x < wn; x += NT) wd[x] = ws[x];
        }
    }
    __syncthreads();                       // the barrier's initialisation is visible to every waiter
    bool ok = rp_mbar_wait(mbar, 0, A.wait_polls);
    // Inspection hook: every copy has landed (phase 0 is complete); phase 1 is completed by nobody,
    // so this second wait gives up after wait_polls polls and the chain takes the time-out path.
    if (ok && A.stall_test && j == 0) ok = rp_mbar_wait(mbar, 1, A.wait_polls);
    return ok;
}

template <int NT, bool WS>
__device__ __forceinline__ void rp_chain_store(const AnnealArgs &A, int j, const char *sm_blob, const int *Wsm, int tid)
{
    const RpDims &dm = A.dm;
    const size_t wn = (size_t)dm.RG * dm.LP;
    const bool w_bulk = WS && ((wn & 3) == 0);
    rp_fence_async_smem();                 // generic-proxy writes to shared memory -> visible to the bulk engine
    __syncthreads();
    if (tid == 0) {
        rp_bulk_s2g(A.blob_dst + (size_t)j * A.bl.bytes, sm_blob, (u32)A.bl.bytes);
        if (w_bulk) {
            int *wd = A.W + (size_t)A.wloc_dst[j] * wn;
            for (size_t off = 0; off < wn * 4; off += 32768) {
                const u32 n = (u32)((wn * 4 - off) < 32768 ? (wn * 4 - off) : 32768);
                rp_bulk_s2g((char *)wd + off, (const char *)Wsm + off, n);
            }
        }
        rp_bulk_commit_wait();
    }
    if (WS && !w_bulk) {
        int *wd = A.W + (size_t)A.wloc_dst[j] * wn;
        for (size_t x = tid; x < wn; x += NT) wd[x] = Wsm[x];
    }
}
