// Fixed-row population annealing (Algorithm 3 of the paper): the per-level chain kernel
// (K5: GuidedProposal, feasibility, IncrementalScore, Metropolis), the level barrier
// (K6 incumbent update + K7 Boltzmann weights and systematic resampling) and the final
// validation (K8).
//
// Mapping.  One CTA runs one chain for all K steps of a level.  The chain's small state
// (assignment, cell statistics, per-row-shard costs, shard work) lives in shared memory.
// Its rank-load tensor W[R][G][L][P] lives in shared memory too when it fits beside a
// second CTA on the SM (small windows), else in global memory as slices of L*P ints that a
// member shares with its ancestor until it rewrites them (see AnnealArgs).  The sample demand
// rows q[i][L][P] are shared by all chains and stay L2-resident.
//
// Three chain kernels: warp per candidate (rp_anneal_wpc.cu: rank loads on chip, or L*P <= 512
// with at most 592 members), warp per chain (rp_anneal_warp.cu: every other window whose rank
// loads are slices of the pool and whose ranks are a power of two from 4 to 128), and the
// 128-thread kernel of this file for what is left (other rank counts, chains too large for the
// staging area of the warp-per-chain kernel, private rank-load cells) and for comparison
// (RP_KNOB_CHAIN_KERNEL).
//
// A chain is a sequential process, but three things about it are not:
//  * every random number is a pure function of (step, level, slot), so the proposal words
//    and the accept threshold -log2(u)*T of the next 32 steps are computed by 32 lanes at once;
//  * a proposal depends on the chain state, which changes only when a move is ACCEPTED, so
//    32 lanes evaluate the proposals and feasibility of the next 32 steps against the current
//    state at once; infeasible steps are skipped in bulk, feasible ones are scored in step
//    order, and the speculation is redone only after an acceptance (the result is identical
//    to stepping one by one);
//  * scoring a move is a data-parallel pass over two L*P slices.
// Resampling is folded into the next level's prologue: slot j starts from the terminal
// state of its ancestor in the other population buffer, so no separate gather pass runs.
// The trajectory-best layout of the kernel below (and of the warp-per-chain kernel) is not copied:
// every accepted move is logged (8 bytes) and the level barrier rebuilds the one winning layout from
// the chain's start layout and its log (the warp-per-candidate kernel snapshots the layout instead).
//
// Algorithmic bytes per feasible move: reads 2 W slices + the moved samples' q rows
// ((3 or 4) * L*P*4 bytes), writes 2 W slices when accepted.
#include "rp_level_end.cuh"

struct ChainB {                 // bookkeeping of the chain within this level
    i64 B[3];
    u64 dig;
    int best_step, best_nlog, nlog, failed;
    unsigned fmask;
    int accept;
    i64 n_feas, n_acc, n_imp, n_bytes;      // counters of the level
    int mt[SPEC][2];                        // lengths of the samples each feasible proposal moves
};

// Chain kernel with NT threads per chain: all of them score one candidate at a time (two L*P
// slices of W from global memory plus the moved samples' demand rows, 16-byte loads into
// registers); the leading warp rebuilds the score and decides.
template <int NT, int MINB, bool SL, bool ALIAS>
__global__ void __launch_bounds__(NT, MINB)
k_anneal_level(const AnnealArgs A)
{
    const RpDims &dm = A.dm;
    extern __shared__ __align__(16) unsigned char smraw[];
    const size_t wn = (size_t)dm.RG * dm.LP;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;
    char *sm_blob = (char *)smraw;
    char *sm_static = sm_blob + A.bl.bytes;
    int *scratch = (int *)(sm_static + A.sl.bytes);
    // Per-cell caches of the proposal keys (attention cost of the cell, cost and attention part of its
    // row-shard).  With one cell per row-shard (every DP slot its own shard) they equal the row-shard
    // arrays of the blob; ALIAS then uses those arrays themselves and keeps no copy (chosen where the
    // shared memory saved lets one more chain be resident per SM).
    i64 *attkey = (i64 *)(scratch + 2 * slice_pad);
    i64 *Jcell = attkey + dm.K;
    i64 *Acell = Jcell + dm.K;
    i64 *red = ALIAS ? attkey : Acell + dm.K;
    StepRec *recs = (StepRec *)(red + 2 * (NT / 32));
    ChainB *chain = (ChainB *)(recs + SPEC);
    u64 *mbar = (u64 *)(chain + 1);
    MoveS *mvs = (MoveS *)(mbar + 1);
    int *spare = (int *)(mvs + SPEC);                       // [RG] slice mode: free slice set aside for each row-shard
    unsigned char *own = (unsigned char *)(spare + (SL ? dm.RG : 0));   // [RG] this chain is the only holder of the row-shard's slice

    u64 *Q = (u64 *)(sm_blob + A.bl.off_Q);
    i64 *Esum = (i64 *)(sm_blob + A.bl.off_Esum);
    i64 *Afx = (i64 *)(sm_blob + A.bl.off_Afx);
    i64 *Jfx = (i64 *)(sm_blob + A.bl.off_Jfx);
    i64 *U = (i64 *)(sm_blob + A.bl.off_U);
    i64 *Sc = (i64 *)(sm_blob + A.bl.off_S);
    int *T = (int *)(sm_blob + A.bl.off_T);
    int *cnt = (int *)(sm_blob + A.bl.off_cnt);
    unsigned short *cell_of = (unsigned short *)(sm_blob + A.bl.off_cell);
    if (ALIAS) { attkey = Afx; Jcell = Jfx; Acell = Afx; }
    int *wtab = (int *)(sm_blob + (SL ? A.bl.off_wtab : 0));          // slice mode: row-shard -> slice of the pool
    const int *dpl = (const int *)(sm_static + A.sl.off_dpl);
    const int *dpo = (const int *)(sm_static + A.sl.off_dpo);
    const int *tt = A.sl.t_staged ? (const int *)(sm_static + A.sl.off_t) : A.t;
    const unsigned short *rg_of = (const unsigned short *)(sm_static + A.sl.off_rg);
    const unsigned short *g_of = (const unsigned short *)(sm_static + A.sl.off_g);
    const unsigned short *rowbase = (const unsigned short *)(sm_static + A.sl.off_row);
    RpSmemState st = { cell_of, T, Q, cnt, Esum, Afx, U };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int j = blockIdx.x;
    // (clamped: after a level that gave up on a wait the table is stale, and the cell look-up below runs
    // before this chain has seen the status word)
    const int src = min(max(A.anc[j], 0), A.Ppop - 1);
    const bool identity_edp = (dm.G == dm.D);
    const int dst_cell = SL ? 0 : A.wloc_dst[j];
    const int src_cell = SL ? 0 : rp_src_cell(A, src, j);
    int *Wj = A.W + (size_t)dst_cell * wn;

    const bool vec = (dm.P >= 4) && (dm.P <= 128) && ((dm.P & (dm.P - 1)) == 0);
    const i64 aC = dm.asum * dm.C, bS = dm.bsum;

    // An earlier level of this call gave up on a wait: its barrier did not run, so the ancestor
    // tables are stale.  Every later chain does nothing but take its ticket.
    if (tid == 0) chain->failed = __ldcg(&A.status[RP_SW_TIMEOUT]) ? 2 : 0;
    __syncthreads();
    if (!chain->failed) {
        const bool landed = rp_chain_load<NT, false>(A, src, j, sm_blob, sm_static, nullptr, mbar, tid, src_cell, dst_cell);
        if (tid == 0 && src_cell != dst_cell)              // bytes of the W gather (counted here: off the level's tail)
            atomicAdd((u64 *)&A.counters[5], (u64)2 * dm.RG * dm.LP * 4);
        if (!landed) chain->failed = 1;
    }
    __syncthreads();
    if (chain->failed) {
        // A bounded wait ran out (1), or an earlier level's did (2): raise the status word, store
        // nothing, and still take the ticket so that the arrival counter stays consistent.
        if (tid == 0 && chain->failed == 1) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
        rp_finish_level(A, tid, NT, smraw, A.smem_bytes);
        return;
    }
    if (!ALIAS)
        for (int c = tid; c < dm.K; c += NT) {
            attkey[c] = aC * (i64)T[c] + bS * (i64)Q[c];
            Jcell[c] = Jfx[rg_of[c]];
            Acell[c] = Afx[rg_of[c]];
        }
    if (tid == 0) {
        chain->B[0] = Sc[0]; chain->B[1] = Sc[1]; chain->B[2] = Sc[2];
        chain->dig = 0; chain->best_step = 0; chain->best_nlog = 0; chain->nlog = 0;
        chain->n_feas = 0; chain->n_acc = 0; chain->n_imp = 0; chain->n_bytes = 0;
    }
    if (SL) {
        // A slice that only this member holds when the level starts is rewritten in place; a shared
        // one is left at its first rewrite for this chain's spare slice of that row-shard (entry
        // j*RG + rg of the free list, which holds at least RG slices per member).  Holder counts are
        // only read here: nobody gains a slice during a level, and nobody who has left one reads it again.
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

    for (int kb = 0; kb < A.steps; kb += SPEC) {
        const int nb = min(SPEC, A.steps - kb);
        if (tid < nb) recs[tid] = rp_make_step_rec(A, A.level, A.tau, (u32)(kb + tid), (u32)j);
        __syncthreads();
        int pos = 0;
        while (pos < nb) {
            if (warp == 0) {
                bool ok = false;
                if (lane >= pos && lane < nb) {
                    MoveS m;
                    int ti, t2;
                    ok = rp_propose_len(dm, view, recs[lane], m, ti, t2);
                    if (ok) { mvs[lane] = m; chain->mt[lane][0] = ti; chain->mt[lane][1] = t2; }
                }
                const unsigned fm = __ballot_sync(0xffffffffu, ok);
                if (lane == 0) { chain->fmask = fm; chain->accept = 0; }
            }
            __syncthreads();
            unsigned fmask = chain->fmask;
            int next_pos = nb;
            while (fmask) {
                const int ls = __ffs(fmask) - 1;
                fmask &= fmask - 1;
                const MoveS m = mvs[ls];
                const bool swap = !m.reloc;
                const int rg1 = rg_of[m.c1], rg2 = rg_of[m.c2];
                const bool touchW = (rg1 != rg2);
                i64 e1 = 0, e2 = 0;
                if (touchW) {
                    const int *qi = A.q + (size_t)m.i * dm.LP;
                    const int *q2 = swap ? A.q + (size_t)m.i2 * dm.LP : nullptr;
                    const int *w1 = SL ? A.W + (size_t)wtab[rg1] * dm.LP : Wj + (size_t)rg1 * dm.LP;
                    const int *w2 = SL ? A.W + (size_t)wtab[rg2] * dm.LP : Wj + (size_t)rg2 * dm.LP;
                    const int P = dm.P, LP = dm.LP;
                    if (vec) {
                        RpSliceRegs<2> regs;
                        for (int base = 0; base < (LP >> 2); base += 2 * NT) {
                            rp_slices_load<2, NT>(regs, base, LP >> 2, (const int4 *)qi, (const int4 *)q2, (const int4 *)w1,
                                                  (const int4 *)w2, tid);
                            rp_slices_reduce<2, NT>(regs, base, LP >> 2, P >> 2, (int4 *)scratch, (int4 *)(scratch + slice_pad),
                                                    tid, e1, e2);
                        }
                    } else {
                        for (int x = tid; x < LP; x += NT) {
                            int d = __ldg(qi + x);
                            if (swap) d -= __ldg(q2 + x);
                            scratch[x] = w1[x] - d;
                            scratch[slice_pad + x] = w2[x] + d;
                        }
                        __syncthreads();
                        for (int l = warp; l < dm.L; l += NT / 32) {
                            int v1 = 0, v2 = 0;
                            for (int p = lane; p < P; p += 32) {
                                v1 = max(v1, scratch[l * P + p]);
                                v2 = max(v2, scratch[slice_pad + l * P + p]);
                            }
                            for (int o = 16; o; o >>= 1) {
                                v1 = max(v1, __shfl_xor_sync(0xffffffffu, v1, o));
                                v2 = max(v2, __shfl_xor_sync(0xffffffffu, v2, o));
                            }
                            if (lane == 0) { e1 += v1; e2 += v2; }
                        }
                    }
                    e1 = warp_sum_i64(e1);
                    e2 = warp_sum_i64(e2);
                    if (lane == 0) { red[2 * warp] = e1; red[2 * warp + 1] = e2; }
                    __syncthreads();
                    if (warp == 0) {
                        e1 = 0; e2 = 0;
                        for (int w = 0; w < NT / 32; ++w) { e1 += red[2 * w]; e2 += red[2 * w + 1]; }
                    }
                }
                if (warp == 0) {
                    const int c1 = m.c1, c2 = m.c2;
                    const int g1 = g_of[c1], g2 = g_of[c2];
                    i64 n0 = 0, n1 = 0, n2 = 0, A1 = 0, A2 = 0, J1n = 0, J2n = 0, U1n = 0, U2n = 0;
                    i64 Ta = 0, Qa = 0, Tb = 0, Qb = 0;
                    int fb0 = 0, fb2 = 0;
                    if (lane == 0) {
                        const i64 S0 = Sc[0], S1 = Sc[1], S2 = Sc[2];
                        const i64 ti = chain->mt[ls][0], t2 = chain->mt[ls][1];
                        Ta = (i64)T[c1] - ti + t2; Qa = (i64)Q[c1] - ti * ti + t2 * t2;
                        Tb = (i64)T[c2] + ti - t2; Qb = (i64)Q[c2] + ti * ti - t2 * t2;
                        if (!touchW) { e1 = Esum[rg1]; e2 = e1; }
                        if (identity_edp) { A1 = aC * Ta + bS * Qa; A2 = aC * Tb + bS * Qb; }
                        else {
                            A1 = rp_attention(dm, st, dpl, dpo, rowbase[c1] / dm.D, g1, c1, Ta, Qa, c2, Tb, Qb);
                            A2 = touchW ? rp_attention(dm, st, dpl, dpo, rowbase[c2] / dm.D, g2, c1, Ta, Qa, c2, Tb, Qb) : A1;
                        }
                        const i64 J1o = Jfx[rg1], J2o = Jfx[rg2];
                        J1n = A1 + dm.EC * e1; J2n = touchW ? A2 + dm.EC * e2 : J1n;
                        const i64 dJ1 = J1n - J1o, dJ2 = touchW ? J2n - J2o : 0;
                        const i64 U1o = U[g1], U2o = U[g2];
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
                    if (fb & 1) {
                        i64 v = 0;
                        for (int g = lane; g < dm.G; g += 32) if (g != g1 && g != g2 && U[g] > v) v = U[g];
                        v = warp_max_i64(v);
                        if (lane == 0 && v > n0) n0 = v;
                    }
                    if (fb & 2) {
                        i64 v = 0;
                        for (int rg = lane; rg < dm.RG; rg += 32) if (rg != rg1 && rg != rg2 && Jfx[rg] > v) v = Jfx[rg];
                        v = warp_max_i64(v);
                        if (lane == 0 && v > n2) n2 = v;
                    }
                    if (lane == 0) {
                        const StepRec rr = recs[ls];
                        const i64 Ecur = Sc[3];
                        bool acc = rp_lex_less(n0, n1, n2, Sc[0], Sc[1], Sc[2]);
                        const i64 en = rp_energy(n0, n1, n2);
                        if (!acc) {
                            if (en <= Ecur || (rr.flags & 4u)) acc = true;
                            else {
                                const u64 M = (u64)(Ecur > dm.SC ? Ecur : dm.SC);
                                const u64 bh = __umul64hi(rr.thr, M), bl = rr.thr * M;
                                acc = (bh >> 31) ? true : ((u64)(en - Ecur) < ((bh << 32) | (bl >> 32)));
                            }
                        }
                        chain->n_feas += 1;
                        if (touchW) chain->n_bytes += (i64)((swap ? 4 : 3) + (acc ? 2 : 0)) * dm.LP * 4;
                        if (acc) {
                            chain->n_acc += 1;
                            if (SL && touchW) {
                                // Where the two rewritten slices go: in place when the slice is this chain's
                                // own, else to the spare slice of that row-shard, which then is its own.
                                const int both[2] = { rg1, rg2 };
                                for (int x = 0; x < 2; ++x) {
                                    const int rg = both[x];
                                    if (own[rg]) continue;
                                    if (spare[rg] >= 0) wtab[rg] = spare[rg];
                                    else atomicExch(&A.status[RP_SW_POOL], 1);           // cannot happen: the list has a spare per row-shard
                                    own[rg] = 1;
                                }
                            }
                            const int k = kb + ls;
                            cell_of[m.i] = (unsigned short)c2;
                            if (swap) cell_of[m.i2] = (unsigned short)c1;
                            T[c1] = (int)Ta; Q[c1] = (u64)Qa; T[c2] = (int)Tb; Q[c2] = (u64)Qb;
                            if (!ALIAS) { attkey[c1] = aC * Ta + bS * Qa; attkey[c2] = aC * Tb + bS * Qb; }
                            if (!swap) { cnt[c1] -= 1; cnt[c2] += 1; }
                            Esum[rg1] = e1; Afx[rg1] = A1; Jfx[rg1] = J1n;
                            if (touchW) { Esum[rg2] = e2; Afx[rg2] = A2; Jfx[rg2] = J2n; }
                            if (ALIAS) { }
                            else if (identity_edp) { Jcell[c1] = J1n; Acell[c1] = A1; Jcell[c2] = J2n; Acell[c2] = A2; }
                            else {
                                for (int x = dpo[g1]; x < dpo[g1 + 1]; ++x) { const int c = rowbase[c1] + dpl[x]; Jcell[c] = J1n; Acell[c] = A1; }
                                for (int x = dpo[g2]; x < dpo[g2 + 1]; ++x) { const int c = rowbase[c2] + dpl[x]; Jcell[c] = J2n; Acell[c] = A2; }
                            }
                            U[g1] = U1n; U[g2] = U2n;
                            Sc[0] = n0; Sc[1] = n1; Sc[2] = n2; Sc[3] = en;
                            const u32 second = swap ? (u32)m.i2 : (u32)c2;
                            int nlog = chain->nlog;
                            if (nlog < A.log_cap) logj[nlog] = make_uint2((u32)m.i, second | (swap ? 0u : 0x80000000u));
                            chain->nlog = ++nlog;
                            const u64 code = ((u64)(swap ? 0 : 1) << 63) ^ ((u64)(u32)k << 40) ^ ((u64)(u32)m.i << 20) ^ (u64)second;
                            chain->dig = (chain->dig ^ code) * 0x100000001B3ull;
                            if (rp_lex_less(n0, n1, n2, chain->B[0], chain->B[1], chain->B[2])) {
                                chain->B[0] = n0; chain->B[1] = n1; chain->B[2] = n2;
                                chain->best_step = k + 1; chain->best_nlog = nlog;
                                chain->n_imp += 1;
                            }
                        }
                        chain->accept = acc;
                    }
                }
                __syncthreads();
                const int acc = chain->accept;
                if (acc) {
                    if (touchW) {
                        int *w1 = SL ? A.W + (size_t)wtab[rg1] * dm.LP : Wj + (size_t)rg1 * dm.LP;
                        int *w2 = SL ? A.W + (size_t)wtab[rg2] * dm.LP : Wj + (size_t)rg2 * dm.LP;
                        if (vec) {
                            for (int c = tid; c < (dm.LP >> 2); c += NT) {
                                ((int4 *)w1)[c] = ((const int4 *)scratch)[c];
                                ((int4 *)w2)[c] = ((const int4 *)(scratch + slice_pad))[c];
                            }
                        } else {
                            for (int x = tid; x < dm.LP; x += NT) { w1[x] = scratch[x]; w2[x] = scratch[slice_pad + x]; }
                        }
                    }
                    next_pos = ls + 1;
                    fmask = 0;
                }
                __syncthreads();
            }
            pos = next_pos;
        }
    }

    rp_chain_store<NT, false>(A, j, sm_blob, nullptr, tid);
    if (tid == 0) {
        for (int x = 0; x < 3; ++x) { A.term[3 * (size_t)j + x] = Sc[x]; A.best[3 * (size_t)j + x] = chain->B[x]; }
        A.best_step[j] = chain->best_step;
        A.best_nlog[j] = chain->best_nlog;
        A.digest[j] = chain->dig;
        atomicAdd((u64 *)&A.counters[0], (u64)A.steps);
        atomicAdd((u64 *)&A.counters[1], (u64)chain->n_feas);
        atomicAdd((u64 *)&A.counters[2], (u64)chain->n_acc);
        atomicAdd((u64 *)&A.counters[3], (u64)chain->n_imp);
        atomicAdd((u64 *)&A.counters[4], (u64)chain->n_bytes);
    }
    rp_finish_level(A, tid, NT, smraw, A.smem_bytes);
}

// Thread count and shared-memory plan of the chain kernels.  Windows with L*P <= 512 use the
// warp-per-candidate kernel; larger ones the kernel above with 128 threads (unless the
// warp-per-chain kernel takes the window, see rp_launch_anneal_level).
size_t rp_wpc_smem_bytes(const RpDims &dm, const RpBlob &bl, const RpStatic &sl, int nw, int *w_in_smem);
int rp_wpc_warps(int pop_size);
int rp_launch_anneal_wpc(rp_ctx *c, const AnnealArgs &A);

static bool use_wpc(const RpDims &dm) { return dm.LP <= 512; }
bool rp_uses_wpc(const RpDims &dm) { return use_wpc(dm); }
// Rank loads in global memory are kept as shared slices (see AnnealArgs); the 128-thread kernel
// can also keep one private cell per member (inspection hook; slower wherever resampling replaces
// many members, never faster).  Decided when the row count is known and kept in the dimensions.
bool rp_uses_slices(const RpDims &dm) { return dm.slices != 0; }
int rp_slice_mode(const RpDims &dm, int knob)
{
    if (use_wpc(dm)) return 0;
    return knob == 2 ? 0 : 1;
}

// Blob and table layouts once the row count is known.  Whether the warp-per-candidate kernel keeps
// the rank loads on chip depends on the blob's size, and the blob carries the slice table only when
// they stay in global memory: lay out without the table first, then again if it is needed.
void rp_decide_layouts(rp_ctx *c)
{
    RpDims &dm = c->dm;
    dm.slices = 0;
    rp_make_layouts(dm, &c->bl, &c->sl);
    if (use_wpc(dm)) {
        int ws = 0;
        rp_wpc_smem_bytes(dm, c->bl, c->sl, rp_wpc_warps(c->Ppop), &ws);
        dm.slices = ws ? 0 : 1;
    } else {
        dm.slices = rp_slice_mode(dm, c->knob_slices);
    }
    if (dm.slices) rp_make_layouts(dm, &c->bl, &c->sl);
}

// Slice bookkeeping between two levels: holders of every slice among the members that start the
// next level (member m starts from the terminal table of anc[m]), then the list of free slices,
// ascending within every block of SLICE_BLOCK slices and block after block in the order the blocks
// arrive (so that a member's RG spares are a nearly contiguous piece of the pool).  The second
// kernel leaves the counts at zero for the next round.
#define SLICE_BLOCK 1024
// After a level that gave up on a wait the ancestors were never written: both kernels then leave
// everything as it is (the chains of the remaining levels do nothing either).  Indices are
// checked before they are used, so that a broken table can only raise the status word.
__global__ void k_slice_holders(const char *__restrict__ blobs, RpBlob bl, const int *__restrict__ anc, int RG, int P, int ns,
                                int *__restrict__ ref, int *__restrict__ head, int *__restrict__ status)
{
    if (__ldcg(&status[RP_SW_TIMEOUT])) return;
    const int a = anc[blockIdx.x];
    if ((unsigned)a >= (unsigned)P) { if (threadIdx.x == 0) atomicExch(&status[RP_SW_POOL], 1); return; }
    const int *tab = (const int *)(blobs + (size_t)a * bl.bytes + bl.off_wtab);
    for (int rg = threadIdx.x; rg < RG; rg += blockDim.x) {
        const int s = tab[rg];
        if ((unsigned)s < (unsigned)ns) atomicAdd(&ref[s], 1);
        else atomicExch(&status[RP_SW_POOL], 1);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { head[0] = 0; head[1] = 0; }
}
__global__ void __launch_bounds__(SLICE_BLOCK)
k_slice_free_list(int *__restrict__ ref, int *__restrict__ holders, int n, int *__restrict__ list, int *__restrict__ head,
                  const int *__restrict__ status)
{
    __shared__ int wsum[32];
    __shared__ int base;
    if (__ldcg(&status[RP_SW_TIMEOUT])) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int s = blockIdx.x * SLICE_BLOCK + threadIdx.x;
    const int r = s < n ? ref[s] : 1;
    if (s < n) { holders[s] = r; ref[s] = 0; }
    const bool is_free = (r == 0);
    const unsigned m = __ballot_sync(0xffffffffu, is_free);
    if (lane == 0) wsum[warp] = __popc(m);
    __syncthreads();
    if (warp == 0) {
        int w = wsum[lane];
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += y; }
        wsum[lane] = w;
        if (lane == 31) base = w ? atomicAdd(&head[1], w) : 0;
    }
    __syncthreads();
    if (is_free) list[base + (warp ? wsum[warp - 1] : 0) + __popc(m & ((1u << lane) - 1))] = s;
}

int rp_launch_slice_gc(rp_ctx *c)
{
    const int ns = 2 * c->Ppop * c->dm.RG, nb = (ns + SLICE_BLOCK - 1) / SLICE_BLOCK;
    k_slice_holders<<<c->Ppop, 128, 0, c->stream>>>(c->buf[c->cur].blob, c->bl, c->d_anc, c->dm.RG, c->Ppop, ns, c->d_wcount,
                                                    c->d_wfree_head, c->d_status);
    k_slice_free_list<<<nb, SLICE_BLOCK, 0, c->stream>>>(c->d_wcount, c->d_wref, ns, c->d_wfree, c->d_wfree_head, c->d_status);
    g_rp_launches += 2;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// Resident chains per SM of the 128-thread kernel: six (80 registers) keep the most bytes in
// flight; windows whose rank loads per member pass a megabyte run faster with five (96 registers,
// no spills; their working set misses L2 either way).
static int rp_coop_chains_per_sm(const RpDims &dm)
{
    return ((size_t)dm.RG * dm.LP * sizeof(int) >= (1u << 20)) ? 5 : 6;
}

int rp_anneal_smem_bytes(const rp_ctx *c, int *threads, size_t *bytes)
{
    const RpDims &dm = c->dm;
    if (use_wpc(dm)) {
        int ws = 0;
        const int nw = rp_wpc_warps(c->Ppop);
        *threads = nw * 32;
        *bytes = rp_wpc_smem_bytes(dm, c->bl, c->sl, nw, &ws);
        return ws;
    }
    const int nt = 128;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;
    size_t b = (size_t)c->bl.bytes + c->sl.bytes + sizeof(int) * 2 * slice_pad + sizeof(i64) * (3 * (size_t)dm.K + 2 * (nt / 32)) +
               sizeof(StepRec) * SPEC + sizeof(ChainB) + sizeof(u64) + sizeof(MoveS) * SPEC + (size_t)dm.RG * 5;
    b = (b + 15) & ~(size_t)15;
    // Without the per-cell key caches (possible with one cell per row-shard): taken when it lets
    // more chains be resident per SM than the registers allow anyway.
    const size_t b_alias = b - sizeof(i64) * 3 * (size_t)dm.K;
    const int minb = rp_coop_chains_per_sm(dm);
    const size_t room = 227 * 1024;
    const bool alias = (dm.G == dm.D) && (room / (b + 1024) < (size_t)minb) && (room / (b_alias + 1024) > room / (b + 1024));
    *threads = nt;
    *bytes = alias ? b_alias : b;
    return alias ? 2 : 0;
}

// Philox4x32-10 on the host (first output word): the resampling offset's random word depends only
// on the seed and the level, so the level barrier does not have to compute it.
static u32 host_philox_x(u32 c0, u32 c1, u32 c2, u32 c3, u32 k0, u32 k1)
{
    for (int r = 0; r < 10; ++r) {
        const u64 p0 = (u64)0xD2511F53u * c0, p1 = (u64)0xCD9E8D57u * c2;
        const u32 n0 = (u32)(p1 >> 32) ^ c1 ^ k0, n2 = (u32)(p0 >> 32) ^ c3 ^ k1;
        c0 = n0; c1 = (u32)p1; c2 = n2; c3 = (u32)p0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

int rp_launch_anneal_wpc_all(rp_ctx *c, const AnnealArgs &A, int *done);
int rp_launch_anneal_warp(rp_ctx *c, AnnealArgs &A);

static void fill_args(rp_ctx *c, int level, int n_levels, const rp_anneal_params *prm, u64 rho_q32, u64 guide_q32, AnnealArgs &A)
{
    A.dm = c->dm; A.bl = c->bl; A.sl = c->sl;
    A.t = c->d_t; A.q = c->d_q; A.static_blk = c->d_static;
    const RpPopBuf &s = c->buf[c->cur], &d = c->buf[1 - c->cur];
    A.blob_src = s.blob; A.blob_dst = d.blob;
    A.W = c->d_W; A.wloc_src = c->d_wloc; A.wloc_dst = c->d_wloc_next;
    A.anc = c->d_anc;
    A.level = level; A.steps = prm->steps_per_level; A.log_cap = c->log_cap;
    A.rho_q32 = rho_q32; A.guide_q32 = guide_q32;
    A.key0 = (u32)c->cfg.seed; A.key1 = (u32)(c->cfg.seed >> 32);
    A.resample_x = host_philox_x(0u, (u32)level, 0u, 3u, A.key0, A.key1);
    A.term = c->d_term; A.best = c->d_best; A.best_step = c->d_best_step; A.best_nlog = c->d_best_nlog;
    A.digest = c->d_digest; A.log = c->d_log; A.counters = c->d_counters; A.status = c->d_status;
    A.tau = c->h_levels[level].tau;
    A.cq = c->h_levels[level].cq;
    A.Ppop = c->Ppop;
    A.last = (level == n_levels - 1);
    A.w_on_chip = 0;
    A.slices = rp_uses_slices(c->dm) ? 1 : 0;
    A.wref = c->d_wref; A.wfree = c->d_wfree; A.wfree_head = c->d_wfree_head;
    A.wait_polls = c->knob_wait_polls > 0 ? c->knob_wait_polls : (1 << 22);
    A.stall_test = c->knob_stall;
    A.le_ws_cap = (unsigned)c->knob_le_ws_cap;
    A.lo.done = c->d_done; A.lo.anc_out = c->d_anc_next; A.lo.F = c->d_F;
    A.lo.wloc_out = c->d_wloc; A.lo.scratch = c->d_le_scratch;   // the barrier rewrites the array the level read from
    A.lo.inc_layout = c->d_inc_layout; A.lo.inc_score = c->d_inc_score;
    A.lo.cand_layout = (use_wpc(c->dm) && !rp_uses_warp_chains(c)) ? c->d_cand_layout : nullptr;
    A.lo.inc_slot = c->d_inc_slot;
    A.lo.tr_term = c->d_tr_term; A.lo.tr_best = c->d_tr_best; A.lo.tr_inc = c->d_tr_inc;
    A.lo.tr_best_step = c->d_tr_best_step; A.lo.tr_anc = c->d_tr_anc; A.lo.tr_digest = c->d_tr_digest;
    A.n_levels = n_levels; A.cur0 = c->cur;
    A.levels = (const RpLevelDev *)c->d_levels;
    A.blob_b0 = c->buf[0].blob; A.blob_b1 = c->buf[1].blob;
    A.sync = c->d_sync;
    A.lo.anc_cur = c->d_anc;
    A.bar_timeout_ns = c->knob_wait_polls > 0 ? (u64)c->knob_wait_polls * 1000ull
                                               : 2000000000ull + (u64)prm->steps_per_level * 50000ull;
}

// The levels' schedule integers for the launch that runs all levels (with the random word behind
// each resampling offset, which depends only on the seed and the level).
int rp_upload_levels(rp_ctx *c, int n_levels)
{
    if (n_levels > c->levels_dev_cap) {
        dev_free(c, c->d_levels); c->d_levels = nullptr; c->levels_dev_cap = 0;
        RpLevelDev *d = nullptr;
        RP_TRY(dev_alloc(c, &d, (size_t)n_levels));
        c->d_levels = d; c->levels_dev_cap = n_levels;
    }
    RpLevelDev *h = (RpLevelDev *)malloc(sizeof(RpLevelDev) * n_levels);
    const u32 k0 = (u32)c->cfg.seed, k1 = (u32)(c->cfg.seed >> 32);
    for (int n = 0; n < n_levels; ++n) {
        h[n].tau = c->h_levels[n].tau; h[n].cq = c->h_levels[n].cq;
        h[n].resample_x = host_philox_x(0u, (u32)n, 0u, 3u, k0, k1); h[n].pad = 0;
    }
    const cudaError_t e = cudaMemcpyAsync(c->d_levels, h, sizeof(RpLevelDev) * n_levels, cudaMemcpyHostToDevice, c->stream);
    free(h);            // pageable source: staged before the call returned
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return RP_OK;
}

// Every level of the call in one launch, when the window allows it (*done = 1); see rp_anneal_wpc.cu.
int rp_launch_anneal_all(rp_ctx *c, int n_levels, const rp_anneal_params *prm, u64 rho_q32, u64 guide_q32, int *done)
{
    *done = 0;
    // Automatic: wherever it is possible (lowest latency of a plan).  A launch whose chains wait for
    // one another needs all of them resident at once, so two such launches do not share the SMs: a
    // caller that plans several windows at once on separate streams asks for one launch per level.
    const bool wanted = c->knob_level_launches != 1;
    if (!use_wpc(c->dm) || !wanted || !c->d_levels) return RP_OK;
    AnnealArgs A;
    fill_args(c, 0, n_levels, prm, rho_q32, guide_q32, A);
    return rp_launch_anneal_wpc_all(c, A, done);
}

int rp_launch_anneal_level(rp_ctx *c, int level, int n_levels, const rp_anneal_params *prm, u64 rho_q32, u64 guide_q32)
{
    AnnealArgs A;
    fill_args(c, level, n_levels, prm, rho_q32, guide_q32, A);
    if (rp_uses_slices(c->dm)) RP_TRY(rp_launch_slice_gc(c));
    if (rp_uses_warp_chains(c)) return rp_launch_anneal_warp(c, A);
    if (use_wpc(c->dm)) return rp_launch_anneal_wpc(c, A);
    int nt; size_t smem;
    const bool alias = rp_anneal_smem_bytes(c, &nt, &smem) == 2;
    if (smem > 220 * 1024) return RP_ERR_RANGE;
    A.smem_bytes = (unsigned)smem;
#define COOP_LAUNCH(MINB_, SL_, ID_)                                                                                 \
    do {                                                                                                     \
        if (smem > 32 * 1024)                                                                                \
            RP_CUDA(cudaFuncSetAttribute(k_anneal_level<128, MINB_, SL_, ID_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        k_anneal_level<128, MINB_, SL_, ID_><<<c->Ppop, 128, smem, c->stream>>>(A);                          \
    } while (0)
    const int minb = rp_coop_chains_per_sm(c->dm);
#define COOP_PICK(SL_, ID_)                                  \
    switch (minb) {                                          \
        case 5: COOP_LAUNCH(5, SL_, ID_); break;             \
        default: COOP_LAUNCH(6, SL_, ID_); break;            \
    }
    if (A.slices) { if (alias) { COOP_PICK(true, true) } else { COOP_PICK(true, false) } }
    else { if (alias) { COOP_PICK(false, true) } else { COOP_PICK(false, false) } }
#undef COOP_PICK
#undef COOP_LAUNCH
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// ---------------------------------------------------------------------------------------------
// Validate(x*): every sample in a real cell, no empty cell, no cell over the token cap.
// (Score consistency and non-regression are checked by the caller from a full rescoring.)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
k_validate(const int *__restrict__ layout, const int *__restrict__ t, RpDims dm, int *__restrict__ fill,
           int *__restrict__ cnt, int *__restrict__ status)
{
    const int tid = threadIdx.x;
    for (int c = tid; c < dm.K; c += 1024) { fill[c] = 0; cnt[c] = 0; }
    __syncthreads();
    int bad = 0;
    for (int i = tid; i < dm.N; i += 1024) {
        int c = layout[i];
        if (c < 0 || c >= dm.K) { bad |= 1; continue; }
        atomicAdd(&fill[c], t[i]);
        atomicAdd(&cnt[c], 1);
    }
    __syncthreads();
    for (int c = tid; c < dm.K; c += 1024) {
        if (cnt[c] < 1) bad |= 2;
        if (fill[c] > dm.C) bad |= 4;
    }
    if (bad) atomicOr(&status[RP_SW_VALIDATE], bad);
}

int rp_launch_validate(rp_ctx *c)
{
    int *fill = (int *)c->d_sort_keys;                 // scratch: 2*K ints fit (K <= N)
    k_validate<<<1, 1024, 0, c->stream>>>(c->d_inc_layout, c->d_t, c->dm, fill, fill + c->dm.K, c->d_status);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
