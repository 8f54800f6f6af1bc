// Chain kernel of the population annealing for latency-bound windows (L*P <= 512):
// "warp per candidate".
//
// One CTA of NW warps runs one chain.  The chain's small state arrives as one blob, and
// its rank-load tensor W (when it fits on chip) as a second bulk asynchronous copy, both
// signalled on one mbarrier; they leave the same way.  The random words and accept
// thresholds of the next NW*32 steps are computed one step per thread.  The leading warp
// then evaluates the proposals of the next 32 steps against the current state, one step
// per lane (a proposal depends on the state, and the state changes only when a move is
// accepted).  The feasible ones are scored NW at a time, one candidate per warp, all
// against the same state: each warp builds the two tentative rank-load slices with 16-byte
// loads, reduces the busiest rank per layer with shuffles, rebuilds the exact score and
// takes the Metropolis decision.  The first accepted candidate in step order is committed
// by its warp straight from its registers, and everything speculated after it is discarded
// and redone; if none is accepted the next NW follow.  This is step-for-step the sequential
// chain of Algorithm 3: a later step is only ever scored against the state it would have seen.
//
// Launched once per level (the last CTA to finish runs the level barrier, rp_level_end), or, where
// the rank loads are on chip and every chain is resident at once, once for all levels (PERSIST):
// then the chains meet at an arrival counter after every level, each CTA works out the barrier
// for itself from the reports of all, and a chain that is its own ancestor keeps its state on chip.
#include <string.h>

#include "rp_level_end.cuh"

struct CandS {                  // a feasible proposal and the cell statistics it would leave behind
    MoveS m;
    int pad;
    i64 Ta, Qa, Tb, Qb;         // token count and sum of squares of the source and target cells after the move
    i64 A1, A2;                 // their attention terms (identity shard map only)
};

struct ChainS {                 // bookkeeping of the chain within this level
    i64 B[3];                   // trajectory-best score
    u64 dig;                    // digest of the accepted moves
    int best_step, best_nlog, nlog, failed;
    i64 I[3];                   // incumbent score when the level started
    int has_snap;               // best_lay holds a layout that beats it
};

// Terminal state out of shared memory without waiting for it to land (the caller has fenced the
// shared-memory writes for the bulk engine and synchronised the CTA).
template <int NT, bool WS>
__device__ __forceinline__ void rp_chain_store_async(const AnnealArgs &A, int j, const char *sm_blob, const int *Wsm, int tid)
{
    const RpDims &dm = A.dm;
    const size_t wn = (size_t)dm.RG * dm.LP;
    const bool w_bulk = WS && ((wn & 3) == 0);
    if (tid == 0) {
        rp_bulk_s2g(A.blob_dst + (size_t)j * A.bl.bytes, sm_blob, (u32)A.bl.bytes);
        if (w_bulk) {
            int *wd = A.W + (size_t)A.wloc_dst[j] * wn;
            for (size_t off = 0; off < wn * 4; off += 32768) {
                const u32 n = (u32)((wn * 4 - off) < 32768 ? (wn * 4 - off) : 32768);
                rp_bulk_s2g((char *)wd + off, (const char *)Wsm + off, n);
            }
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    if (WS && !w_bulk) {
        int *wd = A.W + (size_t)A.wloc_dst[j] * wn;
        for (size_t x = tid; x < wn; x += NT) wd[x] = Wsm[x];
    }
}

// Tail of a chain CTA whose bulk stores are still in flight: publish the report, take a ticket,
// wait until the stores have read shared memory (it is about to be reused or released), and let
// the last arrival run the level barrier.
__device__ __forceinline__ void rp_finish_level_async(const AnnealArgs &A, int tid, int nt, unsigned char *ws, size_t ws_bytes)
{
    __shared__ int is_last_a;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(A.lo.done, 1);
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");      // this thread issued them
        is_last_a = (ticket == (int)gridDim.x - 1);
        if (is_last_a) {
            *A.lo.done = 0;
            if (__ldcg(&A.status[RP_SW_TIMEOUT])) is_last_a = 0;            // some chain gave up: no barrier, the call fails
        }
    }
    __syncthreads();
    if (!is_last_a) return;
    __threadfence();
    rp_level_end(A, tid, nt, ws, rp_le_ws_bytes(A, ws_bytes));
}

// Bounded wait of one thread until a counter that the other CTAs of the launch add to has reached
// `target`; false when the time allowed ran out or another chain has raised the time-out word.
__device__ __forceinline__ bool rp_wait_count(const int *ctr, int target, const AnnealArgs &A)
{
    u64 t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (unsigned it = 0;; ++it) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v >= target) return true;
        if ((it & 15u) == 15u) {
            if (__ldcg(&A.status[RP_SW_TIMEOUT])) return false;
            u64 t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            if (t1 - t0 > A.bar_timeout_ns) return false;
        }
    }
}

template <int NW, bool WS, int CH, bool PERSIST>
__global__ void __launch_bounds__(NW * 32, 16 / NW)
k_anneal_wpc(const AnnealArgs A)
{
    constexpr int NT = NW * 32;
    const RpDims &dm = A.dm;
    extern __shared__ __align__(16) unsigned char smraw[];
    const size_t wn = (size_t)dm.RG * dm.LP;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;           // keeps every slice 16-byte aligned
    char *sm_blob = (char *)smraw;
    char *sm_static = sm_blob + A.bl.bytes;
    int *Wsm = (int *)(sm_static + A.sl.bytes);
    int *scratch = Wsm + (WS ? ((wn + 3) & ~(size_t)3) : 0);
    i64 *attkey = (i64 *)(scratch + (size_t)NW * 2 * slice_pad);
    i64 *Jcell = attkey + dm.K;
    i64 *Acell = Jcell + dm.K;
    StepRec *recs = (StepRec *)(Acell + dm.K);
    ChainS *chain = (ChainS *)(recs + NT);
    u64 *mbar = (u64 *)(chain + 1);
    CandS *cand = (CandS *)(mbar + 1);
    int *vote = (int *)(cand + SPEC);                                    // [NW] accept flags of a wave
    int *rnd = vote + NW;                                               // [0] feasible mask, [1] next position
    unsigned short *best_lay = (unsigned short *)(((size_t)(rnd + 2) + 15) & ~(size_t)15);   // [N] trajectory-best layout
    // Rank loads in global memory are kept as shared slices (see AnnealArgs): a free slice set aside
    // for each row-shard, and whether this chain is the only holder of the row-shard's slice.
    constexpr bool SL = !WS;
    int *spare = (int *)(((size_t)(best_lay + dm.N) + 15) & ~(size_t)15);                    // [RG]
    unsigned char *own = (unsigned char *)(spare + (SL ? dm.RG : 0));                        // [RG]
    // One launch for all levels: cumulative weights and ancestors of the level barrier every CTA works out for itself
    u64 *le_F = (u64 *)(((size_t)(own + (SL ? dm.RG : 0)) + 15) & ~(size_t)15);              // [P_pop]
    int *le_anc = (int *)(le_F + (PERSIST ? A.Ppop : 0));                                    // [P_pop]

    u64 *Q = (u64 *)(sm_blob + A.bl.off_Q);
    i64 *Esum = (i64 *)(sm_blob + A.bl.off_Esum);
    i64 *Afx = (i64 *)(sm_blob + A.bl.off_Afx);
    i64 *Jfx = (i64 *)(sm_blob + A.bl.off_Jfx);
    i64 *U = (i64 *)(sm_blob + A.bl.off_U);
    i64 *Sc = (i64 *)(sm_blob + A.bl.off_S);                            // S0, S1, S2, energy
    int *T = (int *)(sm_blob + A.bl.off_T);
    int *cnt = (int *)(sm_blob + A.bl.off_cnt);
    unsigned short *cell_of = (unsigned short *)(sm_blob + A.bl.off_cell);
    int *wtab = (int *)(sm_blob + (SL ? A.bl.off_wtab : 0));             // row-shard -> slice of the pool
    const int *dpl = (const int *)(sm_static + A.sl.off_dpl);
    const int *dpo = (const int *)(sm_static + A.sl.off_dpo);
    const int *tt = A.sl.t_staged ? (const int *)(sm_static + A.sl.off_t) : A.t;
    const unsigned short *rg_of = (const unsigned short *)(sm_static + A.sl.off_rg);
    const unsigned short *g_of = (const unsigned short *)(sm_static + A.sl.off_g);
    const unsigned short *rowbase = (const unsigned short *)(sm_static + A.sl.off_row);
    RpSmemState st = { cell_of, T, Q, cnt, Esum, Afx, U };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int j = blockIdx.x;
    const bool identity_edp = (dm.G == dm.D);
    const bool vec = (dm.P >= 4) && (dm.P <= 128) && ((dm.P & (dm.P - 1)) == 0);
    const i64 aC = dm.asum * dm.C, bS = dm.bsum;
    // A rank load is at most k*C tokens per cell of the row-shard (conservation of the demand
    // rows, token cap), so the sum over layers of the busiest ranks usually fits 32 bits and
    // the warp can add it up with one reduction instruction.
    const bool sum32 = (i64)dm.L * dm.k * dm.C * ((dm.D + dm.G - 1) / dm.G) < (1ll << 31);

    const int P = A.Ppop;
    const int n_levels = PERSIST ? A.n_levels : 1;
    // One launch for all levels: where this member's terminal rank loads go (the two halves of the
    // cells alternate level by level, as they do between launches).
    int half_w = 0, half_r = 0, inc_slot = -1;
    for (int ln = 0; ln < n_levels; ++ln) {
    const int level = PERSIST ? ln : A.level;
    const u64 tau = PERSIST ? A.levels[ln].tau : A.tau;
    const bool last = PERSIST ? (ln == n_levels - 1) : (A.last != 0);

    // The step records of the first batch depend on nothing the previous level wrote: compute
    // them before waiting for it (launched level by level this kernel uses programmatic stream
    // serialisation, so it may start while the previous level's last CTA runs the barrier).
    if (!PERSIST || ln == 0) {
        const int nb0 = min(NT, A.steps);
        if (tid < nb0) recs[tid] = rp_make_step_rec(A, level, tau, (u32)tid, (u32)blockIdx.x);
    }
    int *Wj = WS ? Wsm : A.W;
    if (!PERSIST || ln == 0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // (clamped: after a level that gave up on a wait the table is stale, and the cell look-up below runs
    // before this chain has seen the status word)
    const int src = min(max(A.anc[j], 0), A.Ppop - 1);
    const int dst_cell = SL ? 0 : A.wloc_dst[j];                 // the previous level's barrier wrote it
    const int src_cell = SL ? 0 : rp_src_cell(A, src, j);
    half_w = (dst_cell >= P) ? 1 : 0;
    half_r = (src_cell >= P) ? 1 : 0;
    // the incumbent's score when the level starts (fetched now, beside the loads above; used below)
    i64 inc0 = 0, inc1 = 0, inc2 = 0;
    if (tid == 0) {
        // An earlier level of this call gave up on a wait: its barrier did not run, so the ancestor
        // tables are stale.  Every later chain does nothing but take its ticket.
        chain->failed = __ldcg(&A.status[RP_SW_TIMEOUT]) ? 2 : 0;
        inc0 = A.lo.inc_score[0]; inc1 = A.lo.inc_score[1]; inc2 = A.lo.inc_score[2];
    }
    __syncthreads();

    // ---- prologue: adopt the ancestor's terminal state -------------------------------
    if (!chain->failed) {
        const bool landed = rp_chain_load<NT, WS>(A, src, j, sm_blob, sm_static, Wsm, mbar, tid, src_cell, dst_cell);
        // Bytes of the rank-load gather (counted here: off the level's tail): a copy made because
        // resampling replaced this member by another one's state.  With the rank loads on chip
        // every member's are staged in and out anyway; a member that kept its own state counts
        // as staging, not as gather.
        if (tid == 0 && src_cell != dst_cell)
            atomicAdd((u64 *)&A.counters[(WS && src == j) ? 6 : 5], (u64)2 * dm.RG * dm.LP * 4);
        if (!landed) chain->failed = 1;
    }
    __syncthreads();
    if (chain->failed) {
        // A bounded wait ran out (1), or an earlier level's did (2): raise the status word, store
        // nothing, and still take the ticket so that the arrival counter stays consistent.  The
        // copies this CTA issued have either landed or have been given wait_polls polls to do so.
        if (tid == 0 && chain->failed == 1) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
        if (PERSIST) return;               // the other chains see the status word while they wait and leave as well
        asm volatile("griddepcontrol.launch_dependents;");
        rp_finish_level_async(A, tid, NT, smraw, A.smem_bytes);
        return;
    }
    if (tid == 0) { chain->I[0] = inc0; chain->I[1] = inc1; chain->I[2] = inc2; }
    }
    for (int c = tid; c < dm.K; c += NT) {
        attkey[c] = aC * (i64)T[c] + bS * (i64)Q[c];
        Jcell[c] = Jfx[rg_of[c]];
        Acell[c] = Afx[rg_of[c]];
    }
    if (tid == 0) {
        chain->B[0] = Sc[0]; chain->B[1] = Sc[1]; chain->B[2] = Sc[2];
        chain->dig = 0; chain->best_step = 0; chain->best_nlog = 0; chain->nlog = 0;
        chain->has_snap = 0;
    }
    if (SL) {
        // A slice that only this member holds when the level starts is rewritten in place; a shared
        // one is left at its first rewrite for this chain's spare slice of that row-shard (entry
        // j*RG + rg of the free list, which holds at least RG slices per member).
        const int n_free = A.wfree_head[1];
        for (int rg = tid; rg < dm.RG; rg += NT) {
            const bool mine = (__ldg(&A.wref[wtab[rg]]) == 1);
            own[rg] = mine ? 1 : 0;
            spare[rg] = mine ? -1 : ((size_t)j * dm.RG + rg < (size_t)n_free ? __ldg(&A.wfree[(size_t)j * dm.RG + rg]) : -1);
        }
    }
    __syncthreads();

        uint2 *logj = A.log + (size_t)j * A.log_cap;
        const RpChainView view = { cell_of, T, cnt, tt, attkey, Jcell, Acell };
        int *my_s1 = scratch + (size_t)warp * 2 * slice_pad, *my_s2 = my_s1 + slice_pad;
        int proposer = 0;                                           // warp that evaluates the next proposals
        i64 w_feas = 0, w_acc = 0, w_imp = 0, w_bytes = 0;          // this warp's share of the counters (lane 0)

        for (int kb = 0; kb < A.steps; kb += NT) {
            const int nb = min(NT, A.steps - kb);
            if (kb > 0 && tid < nb) recs[tid] = rp_make_step_rec(A, level, tau, (u32)(kb + tid), (u32)j);
            __syncthreads();

            int pos = 0;
            while (pos < nb) {
                // ---- proposals of steps kb+pos .. kb+pos+31 against the current state, one per lane,
                // with the part of the scoring that needs only the cell statistics.  The warp that
                // proposes is the one after the last winner, whose own warp is still writing the
                // score-side state of its move (nothing read here).
                if (warp == proposer) {
                    bool ok = false;
                    if (pos + lane < nb) {
                        CandS cd;
                        ok = rp_propose(dm, view, recs[pos + lane], cd.m);
                        if (ok) {
                            const bool swap = !cd.m.reloc;
                            const i64 ti = tt[cd.m.i], t2 = swap ? tt[cd.m.i2] : 0;
                            cd.pad = 0;
                            cd.Ta = (i64)T[cd.m.c1] - ti + t2; cd.Qa = (i64)Q[cd.m.c1] - ti * ti + t2 * t2;
                            cd.Tb = (i64)T[cd.m.c2] + ti - t2; cd.Qb = (i64)Q[cd.m.c2] + ti * ti - t2 * t2;
                            cd.A1 = aC * cd.Ta + bS * cd.Qa; cd.A2 = aC * cd.Tb + bS * cd.Qb;
                            cand[lane] = cd;
                        }
                    }
                    const unsigned fm = __ballot_sync(0xffffffffu, ok);
                    if (lane == 0) rnd[0] = (int)fm;
                }
                __syncthreads();
                unsigned fmask = (unsigned)rnd[0];
                int next_pos = min(pos + SPEC, nb);
                while (fmask) {
                    // ---- one wave: the next NW feasible steps, one per warp, same base state ----
                    unsigned f = fmask;
                    for (int w = 0; w < warp; ++w) f &= f - 1;
                    const int my = f ? (__ffs(f) - 1) : -1;
                    // results of this warp's candidate stay in lane 0's registers until the vote
                    MoveS m;
                    m.reloc = 0; m.i = 0; m.i2 = -1; m.c1 = 0; m.c2 = 0;
                    int rg1 = 0, rg2 = 0, g1 = 0, g2 = 0;
                    bool touchW = false, acc = false;
                    i64 e1 = 0, e2 = 0, A1 = 0, A2 = 0, J1n = 0, J2n = 0, U1n = 0, U2n = 0;
                    i64 n0 = 0, n1 = 0, n2 = 0, en = 0, Ta = 0, Qa = 0, Tb = 0, Qb = 0, my_bytes = 0;
                    if (my >= 0) {
                        m = cand[my].m;
                        const bool swap = !m.reloc;
                        const int c1 = m.c1, c2 = m.c2;
                        rg1 = rg_of[c1]; rg2 = rg_of[c2];
                        g1 = g_of[c1]; g2 = g_of[c2];
                        touchW = (rg1 != rg2);
                        const int *qi = A.q + (size_t)m.i * dm.LP;
                        const int *q2 = swap ? A.q + (size_t)m.i2 * dm.LP : nullptr;
                        const int *w1 = Wj + (size_t)(SL ? wtab[rg1] : rg1) * dm.LP, *w2 = Wj + (size_t)(SL ? wtab[rg2] : rg2) * dm.LP;
                        const int nchunks = dm.LP >> 2;
                        RpSliceRegs<CH> regs;
                        // (a) put the loads of the two slices and the demand rows in flight
                        if (touchW && vec)
                            rp_slices_load<CH, 32>(regs, 0, nchunks, (const int4 *)qi, (const int4 *)q2, (const int4 *)w1,
                                                   (const int4 *)w2, lane);
                        // (b) tentative slices, busiest rank per layer, sum over layers
                        if (touchW) {
                            if (vec) {
                                rp_slices_reduce<CH, 32>(regs, 0, nchunks, dm.P >> 2, (int4 *)my_s1, (int4 *)my_s2, lane, e1, e2);
                                for (int base = CH * 32; base < nchunks; base += CH * 32) {
                                    rp_slices_load<CH, 32>(regs, base, nchunks, (const int4 *)qi, (const int4 *)q2,
                                                           (const int4 *)w1, (const int4 *)w2, lane);
                                    rp_slices_reduce<CH, 32>(regs, base, nchunks, dm.P >> 2, (int4 *)my_s1, (int4 *)my_s2, lane, e1, e2);
                                }
                            } else {
                                for (int x = lane; x < dm.LP; x += 32) {
                                    int d = __ldg(qi + x);
                                    if (swap) d -= __ldg(q2 + x);
                                    my_s1[x] = w1[x] - d;
                                    my_s2[x] = w2[x] + d;
                                }
                                __syncwarp();
                                for (int l = 0; l < dm.L; ++l) {
                                    int v1 = 0, v2 = 0;
                                    for (int p = lane; p < dm.P; p += 32) {
                                        v1 = max(v1, my_s1[l * dm.P + p]);
                                        v2 = max(v2, my_s2[l * dm.P + p]);
                                    }
                                    for (int o = 16; o; o >>= 1) {
                                        v1 = max(v1, __shfl_xor_sync(0xffffffffu, v1, o));
                                        v2 = max(v2, __shfl_xor_sync(0xffffffffu, v2, o));
                                    }
                                    if (lane == 0) { e1 += v1; e2 += v2; }
                                }
                            }
                            if (sum32) {
                                e1 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)e1);
                                e2 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)e2);
                            } else {
                                e1 = warp_sum_i64(e1);
                                e2 = warp_sum_i64(e2);
                            }
                        }
                        // (c) the part of the new score that does not need the rank loads
                        i64 S0 = 0, S1 = 0, S2 = 0, Ecur = 0, J1o = 0, J2o = 0, U1o = 0, U2o = 0;
                        u64 thr = 0;
                        u32 rflags = 0;
                        if (lane == 0) {
                            S0 = Sc[0]; S1 = Sc[1]; S2 = Sc[2]; Ecur = Sc[3];
                            const StepRec rr = recs[pos + my];
                            thr = rr.thr; rflags = rr.flags;
                            const CandS &cd = cand[my];
                            Ta = cd.Ta; Qa = cd.Qa; Tb = cd.Tb; Qb = cd.Qb;
                            if (identity_edp) { A1 = cd.A1; A2 = cd.A2; }
                            else {
                                A1 = rp_attention(dm, st, dpl, dpo, rowbase[c1] / dm.D, g1, c1, Ta, Qa, c2, Tb, Qb);
                                A2 = touchW ? rp_attention(dm, st, dpl, dpo, rowbase[c2] / dm.D, g2, c1, Ta, Qa, c2, Tb, Qb) : A1;
                            }
                            J1o = Jfx[rg1]; J2o = Jfx[rg2];
                            U1o = U[g1]; U2o = U[g2];
                        }
                        // (d) exact new score and the Metropolis decision
                        int fb0 = 0, fb2 = 0;
                        if (lane == 0) {
                            if (!touchW) { e1 = Esum[rg1]; e2 = e1; }
                            J1n = A1 + dm.EC * e1; J2n = touchW ? A2 + dm.EC * e2 : J1n;
                            const i64 dJ1 = J1n - J1o, dJ2 = touchW ? J2n - J2o : 0;
                            if (g1 == g2) { U1n = U1o + dJ1 + dJ2; U2n = U1n; }
                            else { U1n = U1o + dJ1; U2n = U2o + dJ2; }
                            n1 = S1 + dJ1 + dJ2;
                            {
                                const i64 newmax = U1n > U2n ? U1n : U2n, oldmax = U1o > U2o ? U1o : U2o;
                                if (newmax >= S0) n0 = newmax;
                                else if (oldmax < S0) n0 = S0;
                                else { n0 = newmax; fb0 = 1; }
                            }
                            {
                                const i64 newmax = J1n > J2n ? J1n : J2n, oldmax = J1o > J2o ? J1o : J2o;
                                if (newmax >= S2) n2 = newmax;
                                else if (oldmax < S2) n2 = S2;
                                else { n2 = newmax; fb2 = 1; }
                            }
                        }
                        const int fb = __shfl_sync(0xffffffffu, fb0 | (fb2 << 1), 0);
                        if (fb & 1) {       // the previous maximum sat on a changed entry and fell: rescan
                            i64 v = 0;
                            for (int g = lane; g < dm.G; g += 32) if (g != g1 && g != g2 && U[g] > v) v = U[g];
                            v = warp_max_nonneg_i64(v);
                            if (lane == 0 && v > n0) n0 = v;
                        }
                        if (fb & 2) {
                            i64 v = 0;
                            for (int rg = lane; rg < dm.RG; rg += 32) if (rg != rg1 && rg != rg2 && Jfx[rg] > v) v = Jfx[rg];
                            v = warp_max_nonneg_i64(v);
                            if (lane == 0 && v > n2) n2 = v;
                        }
                        if (lane == 0) {
                            acc = rp_lex_less(n0, n1, n2, S0, S1, S2);
                            en = rp_energy(n0, n1, n2);
                            if (!acc) {
                                if (en <= Ecur || (rflags & 4u)) acc = true;
                                else {
                                    const u64 M = (u64)(Ecur > dm.SC ? Ecur : dm.SC);
                                    const u64 bh = __umul64hi(thr, M), bl = thr * M;
                                    acc = (bh >> 31) ? true : ((u64)(en - Ecur) < ((bh << 32) | (bl >> 32)));
                                }
                            }
                            my_bytes = touchW ? (i64)((swap ? 4 : 3) + (acc ? 2 : 0)) * dm.LP * 4 : 0;
                            vote[warp] = acc;
                        }
                    }
                    __syncthreads();
                    const int wave = min(NW, __popc(fmask));
                    int win = -1;
    #pragma unroll
                    for (int w = NW - 1; w >= 0; --w) if (w < wave && vote[w]) win = w;
                    if (my >= 0 && lane == 0 && (win < 0 || warp <= win)) { w_feas += 1; w_bytes += my_bytes; }
                    if (win >= 0) {
                        // commit, first half: what the next proposals read (cells, their statistics and keys)
                        if (warp == win && lane == 0) {
                            const bool swap = !m.reloc;
                            const int c1 = m.c1, c2 = m.c2;
                            cell_of[m.i] = (unsigned short)c2;
                            if (swap) cell_of[m.i2] = (unsigned short)c1;
                            T[c1] = (int)Ta; Q[c1] = (u64)Qa; T[c2] = (int)Tb; Q[c2] = (u64)Qb;
                            if (identity_edp) { attkey[c1] = A1; attkey[c2] = A2; }      // the same expression
                            else { attkey[c1] = aC * Ta + bS * Qa; attkey[c2] = aC * Tb + bS * Qb; }
                            if (!swap) { cnt[c1] -= 1; cnt[c2] += 1; }
                            if (identity_edp) { Jcell[c1] = J1n; Acell[c1] = A1; Jcell[c2] = J2n; Acell[c2] = A2; }
                            else {
                                for (int x = dpo[g1]; x < dpo[g1 + 1]; ++x) { const int c = rowbase[c1] + dpl[x]; Jcell[c] = J1n; Acell[c] = A1; }
                                for (int x = dpo[g2]; x < dpo[g2 + 1]; ++x) { const int c = rowbase[c2] + dpl[x]; Jcell[c] = J2n; Acell[c] = A2; }
                            }
                            rnd[1] = pos + my + 1;
                        }
                        fmask = 0;
                    } else {
                        for (int w = 0; w < wave; ++w) fmask &= fmask - 1;
                    }
                    __syncthreads();
                    if (win >= 0) {
                        next_pos = rnd[1];
                        proposer = win + 1 == NW ? 0 : win + 1;
                        // commit, second half, by the winner's warp while another warp proposes: rank
                        // loads, row-shard and shard costs, score, move log and trajectory best (read
                        // again only after the block-wide barrier that follows the proposals)
                        if (warp == win) {
                            const bool swap = !m.reloc;
                            if (touchW) {
                                if (SL) {      // where the two rewritten slices go: in place when they are this chain's own, else to the spares
                                    if (lane == 0) {
                                        const int both[2] = { rg1, rg2 };
                                        for (int x = 0; x < 2; ++x) {
                                            const int rg = both[x];
                                            if (own[rg]) continue;
                                            if (spare[rg] >= 0) wtab[rg] = spare[rg];
                                            else atomicExch(&A.status[RP_SW_POOL], 1);       // cannot happen: the list has a spare per row-shard
                                            own[rg] = 1;
                                        }
                                    }
                                    __syncwarp();
                                }
                                int *w1 = Wj + (size_t)(SL ? wtab[rg1] : rg1) * dm.LP, *w2 = Wj + (size_t)(SL ? wtab[rg2] : rg2) * dm.LP;
                                if (vec) {
                                    for (int c = lane; c < (dm.LP >> 2); c += 32) {
                                        ((int4 *)w1)[c] = ((const int4 *)my_s1)[c];
                                        ((int4 *)w2)[c] = ((const int4 *)my_s2)[c];
                                    }
                                } else {
                                    for (int x = lane; x < dm.LP; x += 32) { w1[x] = my_s1[x]; w2[x] = my_s2[x]; }
                                }
                            }
                            int snap = 0;
                            if (lane == 0) {
                                const int c2 = m.c2;
                                const int k = kb + pos + my;
                                Esum[rg1] = e1; Afx[rg1] = A1; Jfx[rg1] = J1n;
                                if (touchW) { Esum[rg2] = e2; Afx[rg2] = A2; Jfx[rg2] = J2n; }
                                U[g1] = U1n; U[g2] = U2n;
                                Sc[0] = n0; Sc[1] = n1; Sc[2] = n2; Sc[3] = en;
                                const u32 second = swap ? (u32)m.i2 : (u32)c2;
                                int nlog = chain->nlog;
                                if (nlog < A.log_cap) logj[nlog] = make_uint2((u32)m.i, second | (swap ? 0u : 0x80000000u));
                                chain->nlog = ++nlog;
                                const u64 code = ((u64)(swap ? 0 : 1) << 63) ^ ((u64)(u32)k << 40) ^ ((u64)(u32)m.i << 20) ^ (u64)second;
                                chain->dig = (chain->dig ^ code) * 0x100000001B3ull;
                                w_acc += 1;
                                if (rp_lex_less(n0, n1, n2, chain->B[0], chain->B[1], chain->B[2])) {
                                    chain->B[0] = n0; chain->B[1] = n1; chain->B[2] = n2;
                                    chain->best_step = k + 1; chain->best_nlog = nlog;
                                    w_imp += 1;
                                    snap = rp_lex_less(n0, n1, n2, chain->I[0], chain->I[1], chain->I[2]);
                                }
                            }
                            // a new trajectory best that also beats the incumbent: keep its layout (the first
                            // half of the commit is already in cell_of; the proposing warp only reads it)
                            if (__shfl_sync(0xffffffffu, snap, 0)) {
                                if ((((size_t)cell_of & 15) | ((size_t)dm.N & 7)) == 0) {
                                    const uint4 *sv = (const uint4 *)cell_of;
                                    uint4 *dv = (uint4 *)best_lay;
                                    for (int x = lane; x < (dm.N >> 3); x += 32) dv[x] = sv[x];
                                } else {
                                    for (int x = lane; x < dm.N; x += 32) best_lay[x] = cell_of[x];
                                }
                                if (lane == 0) chain->has_snap = 1;
                            }
                        }
                    }
                }
                pos = next_pos;
            }
        }


    // ---- epilogue: chain report, then the terminal state ---------------------------------------
    // The level barrier reads only the reports (and the layout snapshots), so those go out first
    // with plain stores; launched level by level, the state itself leaves by asynchronous bulk copies
    // that need not have landed before the ticket is taken (the next level starts after this grid
    // has completed).
    if (!PERSIST) rp_fence_async_smem();   // generic-proxy writes to shared memory -> visible to the bulk engine
    __syncthreads();
    if (chain->has_snap) {
        unsigned short *row = A.lo.cand_layout + (size_t)j * dm.N;
        for (int x = tid; x < dm.N; x += NT) row[x] = best_lay[x];
    }
    if (lane == 0) {
        if (w_feas) atomicAdd((u64 *)&A.counters[1], (u64)w_feas);
        if (w_acc) atomicAdd((u64 *)&A.counters[2], (u64)w_acc);
        if (w_imp) atomicAdd((u64 *)&A.counters[3], (u64)w_imp);
        if (w_bytes) atomicAdd((u64 *)&A.counters[4], (u64)w_bytes);
    }
    // reports of this level: one buffer launched level by level, two taken in turn otherwise (a chain
    // that runs ahead must not overwrite what a slower one still reads)
    const size_t rep = PERSIST ? (size_t)(ln & 1) * P : 0;
    if (tid == 0) {
        for (int x = 0; x < 3; ++x) { A.term[3 * (rep + j) + x] = Sc[x]; A.best[3 * (rep + j) + x] = chain->B[x]; }
        A.best_step[rep + j] = chain->best_step;
        A.best_nlog[rep + j] = chain->best_nlog;
        A.digest[rep + j] = chain->dig;
        atomicAdd((u64 *)&A.counters[0], (u64)A.steps);
    }
    if (!PERSIST) {
        rp_chain_store_async<NT, WS>(A, j, sm_blob, Wsm, tid);
        asm volatile("griddepcontrol.launch_dependents;");     // the next level may start its own prologue
        rp_finish_level_async(A, tid, NT, smraw, A.smem_bytes);
        return;
    }

    // ---- one launch for all levels: meet the other chains, publish the state, resample ----------
    // The reports are all the other chains wait for: arrive as soon as they are out.
    __threadfence();
    __syncthreads();
    if (tid == 0) atomicAdd(A.sync, 1);
    // Terminal state with plain stores (whoever descends from this member reads it with plain
    // loads once this member's flag says it is complete): blob into the buffer of this level, rank
    // loads into this member's cell of the half this level writes.
    {
        char *blob_out = (((A.cur0 + ln + 1) & 1) ? A.blob_b1 : A.blob_b0) + (size_t)j * A.bl.bytes;
        const int4 *sb = (const int4 *)sm_blob;
        for (int x = tid; x < (A.bl.bytes >> 4); x += NT) ((int4 *)blob_out)[x] = sb[x];
        int *wd = A.W + ((size_t)half_w * P + j) * wn;
        if ((wn & 3) == 0) for (size_t x = tid; x < (wn >> 2); x += NT) ((int4 *)wd)[x] = ((const int4 *)Wsm)[x];
        else for (size_t x = tid; x < wn; x += NT) wd[x] = Wsm[x];
        if (tid == 0) atomicAdd((u64 *)&A.counters[6], (u64)wn * 4);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(A.sync + 1 + j), "r"(ln + 1) : "memory");
    // while the others finish: the step records of the next level's first batch
    if (!last) {
        const int nb0 = min(NT, A.steps);
        if (tid < nb0) recs[tid] = rp_make_step_rec(A, level + 1, A.levels[ln + 1].tau, (u32)tid, (u32)j);
    }
    if (tid == 0) chain->failed = rp_wait_count(A.sync, (ln + 1) * P, A) ? 0 : 1;
    __syncthreads();
    if (chain->failed) {                     // the wait ran out, or another chain gave up: leave (bounded everywhere)
        if (tid == 0) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
        return;
    }
    // ---- the level barrier, worked out by every CTA for itself (all integer, so all agree) -------
    {
        const i64 *termL = A.term + 3 * rep, *bestL = A.best + 3 * rep;
        __shared__ i64 r0[NW], r1[NW], r2[NW], rmin[NW];
        __shared__ int rj[NW];
        __shared__ u64 rsum[LE_MAX_WARPS];
        __shared__ u64 carry_s;
        __shared__ int win_s;
        // incumbent: the lowest slot among the lexicographically best trajectory-best scores, if it beats it
        i64 b0 = chain->I[0], b1 = chain->I[1], b2 = chain->I[2];
        int bj = 0x7fffffff;
        i64 e_mine = 0x7fffffffffffffffll;
        if (tid < P) {
            const i64 s0 = __ldcg(bestL + 3 * tid), s1 = __ldcg(bestL + 3 * tid + 1), s2 = __ldcg(bestL + 3 * tid + 2);
            if (rp_lex_less(s0, s1, s2, b0, b1, b2)) { b0 = s0; b1 = s1; b2 = s2; bj = tid; }
            e_mine = rp_energy(__ldcg(termL + 3 * tid), __ldcg(termL + 3 * tid + 1), __ldcg(termL + 3 * tid + 2));
        }
        i64 emin = e_mine;
        {
            const u32 hi = (u32)((u64)emin >> 32), mh = __reduce_min_sync(0xffffffffu, hi);
            const u32 ml = __reduce_min_sync(0xffffffffu, hi == mh ? (u32)emin : 0xffffffffu);
            emin = (i64)(((u64)mh << 32) | ml);
        }
        {
            const int srcl = le_lexmin_lane(b0, b1, b2, bj);
            const int sl = srcl < 0 ? 0 : srcl;
            b0 = __shfl_sync(0xffffffffu, b0, sl); b1 = __shfl_sync(0xffffffffu, b1, sl); b2 = __shfl_sync(0xffffffffu, b2, sl);
            bj = __shfl_sync(0xffffffffu, bj, sl);
            if (srcl < 0) bj = 0x7fffffff;
        }
        if (lane == 0) { r0[warp] = b0; r1[warp] = b1; r2[warp] = b2; rj[warp] = bj; rmin[warp] = emin; }
        if (tid == 0) carry_s = 0;
        __syncthreads();
#pragma unroll
        for (int w = 0; w < NW; ++w) emin = rmin[w] < emin ? rmin[w] : emin;
        if (warp == 0) {
            const bool has = lane < NW;
            b0 = has ? r0[lane] : 0; b1 = has ? r1[lane] : 0; b2 = has ? r2[lane] : 0;
            bj = has ? rj[lane] : 0x7fffffff;
            const int srcl = le_lexmin_lane(b0, b1, b2, bj);
            const int sl = srcl < 0 ? 0 : srcl;
            b0 = __shfl_sync(0xffffffffu, b0, sl); b1 = __shfl_sync(0xffffffffu, b1, sl); b2 = __shfl_sync(0xffffffffu, b2, sl);
            bj = __shfl_sync(0xffffffffu, bj, sl);
            if (lane == 0) {
                win_s = -1;
                if (srcl >= 0 && rp_lex_less(b0, b1, b2, chain->I[0], chain->I[1], chain->I[2])) {
                    chain->I[0] = b0; chain->I[1] = b1; chain->I[2] = b2;
                    win_s = bj;                 // that chain stored its trajectory-best layout in its row of cand_layout
                }
            }
        }
        __syncthreads();
        if (win_s >= 0) inc_slot = win_s;
        // Boltzmann weights, cumulative weights, ancestors (not after the last level)
        if (!last) {
            const u64 M = (u64)(emin > dm.SC ? emin : dm.SC);
            le_prefix_weights<1>(P, termL, A.levels[ln].cq, tid, NT, emin, M, le_F, rsum, &carry_s, true, e_mine);
            const u64 Ftot = le_F[P - 1];
            const u64 u0 = (u64)(((unsigned __int128)A.levels[ln].resample_x * Ftot) >> 32);
            if (tid < P) {
                const unsigned __int128 pos = (unsigned __int128)u0 + (unsigned __int128)tid * Ftot;
                int lo = 0, hi = P - 1;
                while (lo < hi) {                       // smallest slot with P * F > pos
                    const int mid = (lo + hi) >> 1;
                    if ((unsigned __int128)P * le_F[mid] > pos) hi = mid; else lo = mid + 1;
                }
                le_anc[tid] = lo;
            }
            __syncthreads();
        }
        // per-level traces (inspection hook), by the first chain
        if (j == 0 && A.lo.tr_term) {
            const size_t o = (size_t)level * P;
            for (int x = tid; x < 3 * P; x += NT) { A.lo.tr_term[o * 3 + x] = __ldcg(termL + x); A.lo.tr_best[o * 3 + x] = __ldcg(bestL + x); }
            for (int x = tid; x < P; x += NT) {
                A.lo.tr_best_step[o + x] = __ldcg(A.best_step + rep + x);
                A.lo.tr_digest[o + x] = __ldcg(A.digest + rep + x);
                if (!last) A.lo.tr_anc[o + x] = le_anc[x];
            }
            if (tid < 3) A.lo.tr_inc[(size_t)level * 3 + tid] = chain->I[tid];
        }
        if (last) {
            // The terminal states are the population as they stand: every member descends from itself,
            // its rank loads sit in the cell this level wrote; the first chain hands the incumbent over.
            if (tid == 0) {
                A.lo.anc_out[j] = j; A.lo.anc_cur[j] = j;
                A.lo.wloc_out[j] = half_w * P + j; A.wloc_dst[j] = half_w * P + j;
            }
            if (j == 0) {
                if (tid < 3) A.lo.inc_score[tid] = chain->I[tid];
                if (inc_slot >= 0) {
                    const unsigned short *row = A.lo.cand_layout + (size_t)inc_slot * dm.N;
                    for (int i = tid; i < dm.N; i += NT) A.lo.inc_layout[i] = __ldcg(row + i);
                }
            }
            return;
        }
        // next level: this slot continues from its ancestor's terminal state; its own is still on chip
        const int anc_j = le_anc[j];
        if (anc_j != j) {
            if (tid == 0) chain->failed = rp_wait_count(A.sync + 1 + anc_j, ln + 1, A) ? 0 : 1;     // its state is complete
            __syncthreads();
            if (chain->failed) {
                if (tid == 0) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
                return;
            }
            const int4 *bs = (const int4 *)((((A.cur0 + ln + 1) & 1) ? A.blob_b1 : A.blob_b0) + (size_t)anc_j * A.bl.bytes);
            for (int x = tid; x < (A.bl.bytes >> 4); x += NT) ((int4 *)sm_blob)[x] = __ldcg(bs + x);
            const int *ws = A.W + ((size_t)half_w * P + anc_j) * wn;
            if ((wn & 3) == 0) for (size_t x = tid; x < (wn >> 2); x += NT) ((int4 *)Wsm)[x] = __ldcg((const int4 *)ws + x);
            else for (size_t x = tid; x < wn; x += NT) Wsm[x] = __ldcg(ws + x);
            if (tid == 0) atomicAdd((u64 *)&A.counters[5], (u64)2 * wn * 4);
        }
        half_r = half_w; half_w ^= 1;
        __syncthreads();
    }
    }
}

// Warps per chain: more warps score more candidates of a round at once (good when few chains
// must hide a lot of latency), fewer warps let more chains be resident per SM.  Register use is
// capped at 128 per thread, so NW warps per chain allow 16/NW chains per SM.
int rp_wpc_warps(int pop_size)
{
    return pop_size <= 2 * 148 ? 8 : 4;
}

// Shared-memory bytes of the warp-per-candidate kernel; *w_in_smem says whether W fits on chip
// while still leaving room for the 16/NW chains per SM that the register budget allows.
size_t rp_wpc_smem_bytes(const RpDims &dm, const RpBlob &bl, const RpStatic &sl, int nw, int *w_in_smem)
{
    const int NT = nw * 32;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;
    size_t b = (size_t)bl.bytes + sl.bytes + sizeof(int) * nw * 2 * slice_pad + sizeof(i64) * 3 * dm.K +
               sizeof(StepRec) * NT + sizeof(ChainS) + sizeof(u64) + sizeof(CandS) * SPEC + sizeof(int) * (nw + 2) +
               16 + ((sizeof(unsigned short) * dm.N + 15) & ~(size_t)15);
    const size_t wbytes = sizeof(int) * ((((size_t)dm.RG * dm.LP) + 3) & ~(size_t)3);
    const size_t per_cta = (size_t)220 * 1024 / (16 / nw);
    *w_in_smem = (b + wbytes <= per_cta);
    if (*w_in_smem) b += wbytes;
    else b += 16 + (size_t)dm.RG * 5;            // spare slices and ownership flags
    return (b + 15) & ~(size_t)15;
}

template <int NW>
static int launch_wpc(rp_ctx *c, const AnnealArgs &A, int ws, size_t smem, int chunks)
{
#define LAUNCH(WS_, CH_)                                                                              \
    do {                                                                                              \
        if (smem > 32 * 1024)                                                                         \
            RP_CUDA(cudaFuncSetAttribute(k_anneal_wpc<NW, WS_, CH_, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        cudaLaunchConfig_t cfg;                                                                       \
        memset(&cfg, 0, sizeof cfg);                                                                  \
        cfg.gridDim = dim3(c->Ppop); cfg.blockDim = dim3(NW * 32);                                    \
        cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;                                          \
        cudaLaunchAttribute at[1];                                                                    \
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                \
        at[0].val.programmaticStreamSerializationAllowed = 1;                                         \
        cfg.attrs = at; cfg.numAttrs = 1;                                                             \
        RP_CUDA(cudaLaunchKernelEx(&cfg, k_anneal_wpc<NW, WS_, CH_, false>, A));                       \
    } while (0)
    if (ws) { if (chunks <= 1) LAUNCH(true, 1); else if (chunks <= 2) LAUNCH(true, 2); else LAUNCH(true, 4); }
    else { if (chunks <= 1) LAUNCH(false, 1); else if (chunks <= 2) LAUNCH(false, 2); else LAUNCH(false, 4); }
#undef LAUNCH
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

int rp_launch_anneal_wpc(rp_ctx *c, const AnnealArgs &A0)
{
    const RpDims &dm = c->dm;
    const int nw = rp_wpc_warps(c->Ppop);
    int ws = 0;
    const size_t smem = rp_wpc_smem_bytes(dm, c->bl, c->sl, nw, &ws);
    AnnealArgs A = A0;
    A.w_on_chip = ws;
    A.slices = ws ? 0 : 1;
    A.smem_bytes = (unsigned)smem;
    if (smem > 220 * 1024) return RP_ERR_RANGE;
    const int chunks = ((dm.LP >> 2) + 31) / 32;
    if (nw == 8) return launch_wpc<8>(c, A, ws, smem, chunks);
    return launch_wpc<4>(c, A, ws, smem, chunks);
}

// One launch for all levels.  Possible when the rank loads live on chip, the population is at most
// one member per thread (the level barrier is worked out by every CTA for itself) and every chain
// can be resident at once (cooperative launch, checked with the occupancy calculator).  *done = 0
// when it is not possible: the caller then launches level by level.
template <int NW, int CH>
static int launch_wpc_all(rp_ctx *c, const AnnealArgs &A, size_t smem, int *done)
{
    auto kern = k_anneal_wpc<NW, true, CH, true>;
    if (smem > 32 * 1024) RP_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0, sms = 0;
    RP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NW * 32, smem));
    RP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, c->device));
    if ((long long)per_sm * sms < c->Ppop) return RP_OK;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(c->Ppop); cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;
    at[0].val.cooperative = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, A);
    if (e == cudaErrorCooperativeLaunchTooLarge) { cudaGetLastError(); return RP_OK; }
    RP_CUDA(e);
    ++g_rp_launches;
    *done = 1;
    return RP_OK;
}

int rp_launch_anneal_wpc_all(rp_ctx *c, const AnnealArgs &A0, int *done)
{
    const RpDims &dm = c->dm;
    *done = 0;
    const int nw = rp_wpc_warps(c->Ppop);
    int ws = 0;
    size_t smem = rp_wpc_smem_bytes(dm, c->bl, c->sl, nw, &ws);
    if (!ws || c->Ppop > nw * 32 || nw != 8) return RP_OK;
    smem += 16 + (size_t)c->Ppop * 12;                      // cumulative weights and ancestors of the level barrier
    if (smem > 220 * 1024) return RP_OK;
    AnnealArgs A = A0;
    A.w_on_chip = 1;
    A.slices = 0;
    A.smem_bytes = (unsigned)smem;
    const int chunks = ((dm.LP >> 2) + 31) / 32;
    if (chunks <= 1) return launch_wpc_all<8, 1>(c, A, smem, done);
    if (chunks <= 2) return launch_wpc_all<8, 2>(c, A, smem, done);
    return launch_wpc_all<8, 4>(c, A, smem, done);
}
