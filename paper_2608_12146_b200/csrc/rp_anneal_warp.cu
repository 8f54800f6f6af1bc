// Chain kernel of the population annealing for windows whose rank loads live in the slice pool
// and whose chains outnumber what the multi-warp kernels keep resident: "warp per chain".
//
// A chain of Algorithm 3 is a sequence of dependent rounds (proposal, the touched rank-load
// slices and demand rows from L2 or HBM, exact rescoring in 64-bit integers, decision), so the
// throughput of a level is the number of chains an SM keeps in flight over the latency of a round.
// Here a chain is a single warp (on the largest window: 23 KB of shared memory, nine to an SM):
//  * the two demand rows and two slices of a candidate (4 * L*P ints) arrive in shared memory by
//    four bulk asynchronous copies on one mbarrier (bounded wait): one trip to memory per
//    candidate and no registers held while it lasts; lane 0 rebuilds the part of the score that
//    needs only the cell statistics in the meantime;
//  * the busiest rank of every layer is found with a lane per layer (no shuffles), and an accepted
//    move is stored straight from the staged copies;
//  * the random words of the next 32 steps, the cells of their candidate samples and those
//    samples' lengths are fetched once per batch, one step per lane, and kept in registers; an
//    accepted move patches the cached cells, so a proposal reads shared memory only;
//  * the assignment itself stays in the chain's blob in global memory (written on acceptance,
//    read once per batch), the chain's small arrays arrive and leave with plain loads and stores,
//    and the level barrier (incumbent, weights, ancestors) is a launch of its own behind the chains.
// Step for step this is the sequential chain: proposals are evaluated against the current state,
// feasible ones are scored in step order, and the speculation is redone after an acceptance.
// Rank loads are slices of the pool shared copy-on-write with the ancestor (see AnnealArgs).
#include <algorithm>

#include "rp_level_end.cuh"

#define WARP_CHAINS_PER_SM 9            // resident chains the register budget is set for
#define WARP_SMEM_OPTIN (208 * 1024)    // dynamic shared memory these kernels may ask for (227 KB per CTA on sm_100a, less their static arrays)

struct CandW { MoveS m; int ti, t2, pad; };          // a feasible proposal and the lengths of the moved samples
struct ChainW {                                      // bookkeeping of the chain within this level
    i64 B[3];
    u64 dig;
    int best_step, best_nlog, nlog, pad;
    i64 n_feas, n_acc, n_imp, n_bytes;               // counters of the level
};

// Shared-memory plan of one chain: the blob's arrays up to the assignment at their blob offsets,
// then the slice table, the static tables, the kernel's own arrays and the staging area.
struct RpWarpLayout {
    int off_wtab, off_static, off_keys, off_recs, off_cand, off_chain, off_spare, off_own, off_mbar, off_stage, bytes;
};

static RpWarpLayout rp_warp_layout(const RpDims &dm, const RpBlob &bl, const RpStatic &sl, bool identity)
{
    RpWarpLayout w;
    size_t o = ((size_t)bl.off_cell + 15) & ~(size_t)15;
    w.off_wtab = (int)o;   o += ((size_t)4 * dm.RG + 15) & ~(size_t)15;
    w.off_static = (int)o; o += sl.bytes;
    w.off_keys = (int)o;   o += identity ? 0 : (size_t)3 * 8 * dm.K;
    w.off_recs = (int)o;   o += sizeof(StepRec) * SPEC;
    w.off_cand = (int)o;   o += sizeof(CandW) * SPEC;
    w.off_chain = (int)o;  o += sizeof(ChainW);
    w.off_spare = (int)o;  o += (size_t)4 * dm.RG;
    w.off_own = (int)o;    o += dm.RG;
    o = (o + 15) & ~(size_t)15;
    w.off_mbar = (int)o;   o += 16;
    o = (o + 127) & ~(size_t)127;
    w.off_stage = (int)o;  o += (size_t)4 * 4 * dm.LP;          // two demand rows and two slices of a candidate
    w.bytes = (int)((o + 15) & ~(size_t)15);
    return w;
}

// What a lane keeps about the step it proposes for: the candidate indices of the step record with
// the cells of the candidate samples (kept in step with the accepted moves) and their lengths.
struct StepRegs {
    u32 flags, bz;
    int i[4];               // samples; for a relocation i[2], i[3] are target cells
    int c[4];               // cell of sample i[x] (i[2], i[3] themselves for a relocation)
    int t[4];               // length of sample i[x] (unused for relocation targets)
};

// GuidedProposal + feasibility of one step (the rule of rp_propose) from the lane's registers.
__device__ __forceinline__ bool rp_propose_regs(const RpDims &dm, const StepRegs &r, const int *T, const int *cnt,
                                                const i64 *attkey, const i64 *Jcell, const i64 *Acell, CandW &cd)
{
    const bool reloc = r.flags & 1u;
    const int ca = r.c[0], cb = r.c[1], xa = r.c[2], xb = r.c[3];
    const u64 Ja = (u64)Jcell[ca], Aa = (u64)Acell[ca];
    const u64 lh = __umul64hi((u64)r.bz, Ja), ll = (u64)r.bz * Ja;
    const u64 rh = Aa >> 32, rl = Aa << 32;
    const bool use_att = (lh < rh) || (lh == rh && ll < rl);
    const i64 *key = use_att ? attkey : Jcell;
    const i64 ka = key[ca], kb = key[cb], ta = key[xa], tb = key[xb];
    const bool src_b = kb > ka, dst_b = tb < ta;
    MoveS &m = cd.m;
    m.reloc = reloc;
    m.i = src_b ? r.i[1] : r.i[0];
    m.c1 = src_b ? cb : ca;
    m.c2 = dst_b ? xb : xa;
    m.i2 = reloc ? -1 : (dst_b ? r.i[3] : r.i[2]);
    const int ti = src_b ? r.t[1] : r.t[0];
    const int t2 = reloc ? 0 : (dst_b ? r.t[3] : r.t[2]);
    cd.ti = ti; cd.t2 = t2; cd.pad = 0;
    if (m.c1 == m.c2) return false;
    if (reloc) return (cnt[m.c1] > 1) && (T[m.c2] + ti <= dm.C);
    return (T[m.c1] - ti + t2 <= dm.C) && (T[m.c2] - t2 + ti <= dm.C);
}

// Scoring pass over a candidate whose two demand rows and two slices have been staged in shared
// memory: W1' = W1 - d and W2' = W2 + d with d = q[i] - q[i2] (relocation: d = q[i]).  A lane takes
// whole layers (layer = lane, lane + 32, ...), so the busiest rank of a layer needs no shuffles;
// the lanes of a quarter warp start at different chunks of their layers, which keeps the 16-byte
// reads off each other's banks.  cpl = 16-byte chunks per layer (a power of two).  Returns the
// two sums over layers of the busiest ranks.
template <int CPL>      // chunks per layer when known at compile time (the loop over them is then unrolled), else 0
__device__ __forceinline__ void rp_warp_staged_score_t(int lane, int L, int cpl_rt, bool sum32, bool swap, const int4 *s_qi,
                                                       const int4 *s_q2, const int4 *s_w1, const int4 *s_w2, i64 &e1, i64 &e2)
{
    const int cpl = CPL ? CPL : cpl_rt;
    int p1 = 0, p2 = 0;
    for (int ly = lane; ly < L; ly += 32) {
        const int base = ly * cpl;
        int m1 = 0, m2 = 0;
#pragma unroll (CPL ? CPL : 4)
        for (int k = 0; k < cpl; ++k) {
            const int c = base + ((k + lane) & (cpl - 1));
            int4 d = s_qi[c];
            if (swap) { const int4 o = s_q2[c]; d.x -= o.x; d.y -= o.y; d.z -= o.z; d.w -= o.w; }
            const int4 a = s_w1[c], b = s_w2[c];
            m1 = max(m1, max(max(a.x - d.x, a.y - d.y), max(a.z - d.z, a.w - d.w)));
            m2 = max(m2, max(max(b.x + d.x, b.y + d.y), max(b.z + d.z, b.w + d.w)));
        }
        if (sum32) { p1 += m1; p2 += m2; }
        else { e1 += m1; e2 += m2; }
    }
    if (sum32) {
        e1 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)p1);
        e2 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)p2);
    } else {
        e1 = warp_sum_i64(e1);
        e2 = warp_sum_i64(e2);
    }
}

__device__ __forceinline__ void rp_warp_staged_score(int lane, int L, int cpl, bool sum32, bool swap, const int4 *s_qi,
                                                     const int4 *s_q2, const int4 *s_w1, const int4 *s_w2, i64 &e1, i64 &e2)
{
    if (cpl == 8) rp_warp_staged_score_t<8>(lane, L, cpl, sum32, swap, s_qi, s_q2, s_w1, s_w2, e1, e2);
    else if (cpl == 4) rp_warp_staged_score_t<4>(lane, L, cpl, sum32, swap, s_qi, s_q2, s_w1, s_w2, e1, e2);
    else rp_warp_staged_score_t<0>(lane, L, cpl, sum32, swap, s_qi, s_q2, s_w1, s_w2, e1, e2);
}

// An accepted move: the two new slices straight from the staged copies to where they now live,
// consecutive lanes storing consecutive 16-byte chunks.
__device__ __forceinline__ void rp_warp_staged_commit(int lane, int nchunks, bool swap, const int4 *s_qi, const int4 *s_q2,
                                                      const int4 *s_w1, const int4 *s_w2, int4 *o1, int4 *o2)
{
#pragma unroll 4
    for (int c = lane; c < nchunks; c += 32) {
        int4 d = s_qi[c];
        if (swap) { const int4 o = s_q2[c]; d.x -= o.x; d.y -= o.y; d.z -= o.z; d.w -= o.w; }
        const int4 a = s_w1[c], b = s_w2[c];
        o1[c] = make_int4(a.x - d.x, a.y - d.y, a.z - d.z, a.w - d.w);
        o2[c] = make_int4(b.x + d.x, b.y + d.y, b.z + d.z, b.w + d.w);
    }
}

// ID: every DP slot is its own shard, so a cell is a row-shard and the per-cell proposal keys are
// the row-shard arrays of the blob themselves.
template <bool ID>
__global__ void __launch_bounds__(32, WARP_CHAINS_PER_SM)
k_anneal_warp(const AnnealArgs A, const RpWarpLayout wl)
{
    const RpDims &dm = A.dm;
    extern __shared__ __align__(16) unsigned char smraw[];
    char *sm = (char *)smraw;
    u64 *Q = (u64 *)(sm + A.bl.off_Q);
    i64 *Esum = (i64 *)(sm + A.bl.off_Esum);
    i64 *Afx = (i64 *)(sm + A.bl.off_Afx);
    i64 *Jfx = (i64 *)(sm + A.bl.off_Jfx);
    i64 *U = (i64 *)(sm + A.bl.off_U);
    i64 *Sc = (i64 *)(sm + A.bl.off_S);                              // S0, S1, S2, energy
    int *T = (int *)(sm + A.bl.off_T);
    int *cnt = (int *)(sm + A.bl.off_cnt);
    int *wtab = (int *)(sm + wl.off_wtab);
    char *sm_static = sm + wl.off_static;
    i64 *attkey = ID ? Afx : (i64 *)(sm + wl.off_keys);
    i64 *Jcell = ID ? Jfx : attkey + dm.K;
    i64 *Acell = ID ? Afx : Jcell + dm.K;
    StepRec *recs = (StepRec *)(sm + wl.off_recs);
    CandW *cand = (CandW *)(sm + wl.off_cand);
    ChainW *chain = (ChainW *)(sm + wl.off_chain);
    int *spare = (int *)(sm + wl.off_spare);
    unsigned char *own = (unsigned char *)(sm + wl.off_own);
    u64 *mbar = (u64 *)(sm + wl.off_mbar);
    int4 *s_qi = (int4 *)(sm + wl.off_stage), *s_q2 = s_qi + (dm.LP >> 2), *s_w1 = s_q2 + (dm.LP >> 2), *s_w2 = s_w1 + (dm.LP >> 2);
    const int *dpl = (const int *)(sm_static + A.sl.off_dpl);
    const int *dpo = (const int *)(sm_static + A.sl.off_dpo);
    const unsigned short *rg_of = (const unsigned short *)(sm_static + A.sl.off_rg);
    const unsigned short *g_of = (const unsigned short *)(sm_static + A.sl.off_g);
    const unsigned short *rowbase = (const unsigned short *)(sm_static + A.sl.off_row);
    RpSmemState st = { nullptr, T, Q, cnt, Esum, Afx, U };

    const int lane = threadIdx.x;
    const int j = blockIdx.x;
    if (__ldcg(&A.status[RP_SW_TIMEOUT])) return;                  // the call has failed already: nothing to do
    const int src = min(max(A.anc[j], 0), A.Ppop - 1);
    const int LP = dm.LP, nchunks = LP >> 2, cpl = dm.P >> 2;      // 16-byte chunks per slice and per layer
    const bool sum32 = (i64)dm.L * dm.k * dm.C * ((dm.D + dm.G - 1) / dm.G) < (1ll << 31);
    // The chain's assignment: the 16-bit array of its blob, read and written through L2.
    unsigned short *cells = (unsigned short *)(A.blob_dst + (size_t)j * A.bl.bytes + A.bl.off_cell);
    u32 phase = 0;
    if (lane == 0) rp_mbar_init(mbar, 1);

    // ---- prologue: the ancestor's terminal state --------------------------------------------
    {
        const char *bsrc = A.blob_src + (size_t)src * A.bl.bytes;
        const int nh = A.bl.off_cell >> 2;
        for (int x = lane; x < nh; x += 32) ((int *)sm)[x] = __ldg((const int *)bsrc + x);
        const unsigned short *cs = (const unsigned short *)(bsrc + A.bl.off_cell);
        const int n4 = dm.N >> 2;
        for (int x = lane; x < n4; x += 32) ((uint2 *)cells)[x] = __ldg((const uint2 *)cs + x);
        for (int i = (n4 << 2) + lane; i < dm.N; i += 32) cells[i] = __ldg(cs + i);
        const int *ts = (const int *)(bsrc + A.bl.off_wtab);
        for (int rg = lane; rg < dm.RG; rg += 32) wtab[rg] = __ldg(ts + rg);
        const int nsb = A.sl.bytes >> 2;
        for (int x = lane; x < nsb; x += 32) ((int *)sm_static)[x] = __ldg((const int *)A.static_blk + x);
    }
    __syncwarp();
    if (!ID)
        for (int c = lane; c < dm.K; c += 32) {
            attkey[c] = dm.asum * dm.C * (i64)T[c] + dm.bsum * (i64)Q[c];
            Jcell[c] = Jfx[rg_of[c]];
            Acell[c] = Afx[rg_of[c]];
        }
    if (lane == 0) {
        chain->B[0] = Sc[0]; chain->B[1] = Sc[1]; chain->B[2] = Sc[2];
        chain->dig = 0; chain->best_step = 0; chain->best_nlog = 0; chain->nlog = 0;
        chain->n_feas = 0; chain->n_acc = 0; chain->n_imp = 0; chain->n_bytes = 0;
    }
    {
        // A slice that only this member holds when the level starts is rewritten in place; a shared
        // one is left at its first rewrite for this chain's spare slice of that row-shard (entry
        // j*RG + rg of the free list, which holds at least RG slices per member).
        const int n_free = A.wfree_head[1];
        for (int rg = lane; rg < dm.RG; rg += 32) {
            const bool mine = (__ldg(&A.wref[wtab[rg]]) == 1);
            own[rg] = mine ? 1 : 0;
            spare[rg] = mine ? -1 : ((size_t)j * dm.RG + rg < (size_t)n_free ? __ldg(&A.wfree[(size_t)j * dm.RG + rg]) : -1);
        }
    }
    __syncwarp();

    for (int kb = 0; kb < A.steps; kb += SPEC) {
        const int nb = min(SPEC, A.steps - kb);
        // ---- the next 32 steps, one per lane: random words, candidate cells and lengths -------
        StepRegs sr;
        sr.flags = 0; sr.bz = 0;
#pragma unroll
        for (int x = 0; x < 4; ++x) { sr.i[x] = -1; sr.c[x] = 0; sr.t[x] = 0; }
        if (lane < nb) {
            const StepRec r = rp_make_step_rec(A, A.level, A.tau, (u32)(kb + lane), (u32)j);
            recs[lane] = r;
            const bool rl = r.flags & 1u;
            sr.flags = r.flags; sr.bz = r.bz;
            sr.i[0] = r.i0; sr.i[1] = r.i1; sr.i[2] = r.i2; sr.i[3] = r.i3;
            sr.c[0] = (int)__ldcg(cells + r.i0); sr.c[1] = (int)__ldcg(cells + r.i1);
            sr.c[2] = rl ? r.i2 : (int)__ldcg(cells + r.i2);
            sr.c[3] = rl ? r.i3 : (int)__ldcg(cells + r.i3);
            sr.t[0] = __ldg(A.t + r.i0); sr.t[1] = __ldg(A.t + r.i1);
            sr.t[2] = rl ? 0 : __ldg(A.t + r.i2);
            sr.t[3] = rl ? 0 : __ldg(A.t + r.i3);
        }
        __syncwarp();
        int pos = 0;
        while (pos < nb) {
            // proposals of steps kb+pos .. kb+nb-1 against the current state, one per lane
            bool ok = false;
            if (lane >= pos && lane < nb) {
                CandW cd;
                ok = rp_propose_regs(dm, sr, T, cnt, attkey, Jcell, Acell, cd);
                if (ok) cand[lane] = cd;
            }
            unsigned fmask = __ballot_sync(0xffffffffu, ok);
            __syncwarp();
            int next_pos = nb;
            while (fmask) {
                const int ls = __ffs(fmask) - 1;
                fmask &= fmask - 1;
                const MoveS m = cand[ls].m;
                const bool swap = !m.reloc;
                const int c1 = m.c1, c2 = m.c2;
                const int rg1 = rg_of[c1], rg2 = rg_of[c2];
                const int g1 = g_of[c1], g2 = g_of[c2];
                const bool touchW = (rg1 != rg2);
                const int4 *w1 = (const int4 *)(A.W + (size_t)wtab[rg1] * LP);
                const int4 *w2 = (const int4 *)(A.W + (size_t)wtab[rg2] * LP);
                if (touchW && lane == 0) {
                    // the candidate's rows and slices into shared memory: one trip, nothing in registers
                    const u32 bytes = (u32)LP * 4u;
                    // (the previous candidate's reads of the staging area are complete: their values were used
                    // before the warp-wide barrier that precedes this point)
                    rp_mbar_expect_tx(mbar, (swap ? 4u : 3u) * bytes);
                    rp_bulk_g2s(s_qi, A.q + (size_t)m.i * LP, bytes, mbar);
                    if (swap) rp_bulk_g2s(s_q2, A.q + (size_t)m.i2 * LP, bytes, mbar);
                    rp_bulk_g2s(s_w1, w1, bytes, mbar);
                    rp_bulk_g2s(s_w2, w2, bytes, mbar);
                }
                // ---- lane 0, while the copies are on their way: the part of the new score that needs
                // only the cell statistics, and the accept bound
                i64 S0 = 0, S1 = 0, S2 = 0, Ecur = 0, Ta = 0, Qa = 0, Tb = 0, Qb = 0, A1 = 0, A2 = 0;
                i64 J1o = 0, J2o = 0, U1o = 0, U2o = 0;
                u64 bound = 0;                      // accept when the energy rises by less than this
                bool always = false;                // the bound does not fit 64 bits, or the threshold is saturated
                if (lane == 0) {
                    S0 = Sc[0]; S1 = Sc[1]; S2 = Sc[2]; Ecur = Sc[3];
                    const i64 ti = cand[ls].ti, t2 = cand[ls].t2;
                    Ta = (i64)T[c1] - ti + t2; Qa = (i64)Q[c1] - ti * ti + t2 * t2;
                    Tb = (i64)T[c2] + ti - t2; Qb = (i64)Q[c2] + ti * ti - t2 * t2;
                    const i64 aC = dm.asum * dm.C, bS = dm.bsum;
                    if (ID) { A1 = aC * Ta + bS * Qa; A2 = aC * Tb + bS * Qb; }
                    else {
                        A1 = rp_attention(dm, st, dpl, dpo, rowbase[c1] / dm.D, g1, c1, Ta, Qa, c2, Tb, Qb);
                        A2 = touchW ? rp_attention(dm, st, dpl, dpo, rowbase[c2] / dm.D, g2, c1, Ta, Qa, c2, Tb, Qb) : A1;
                    }
                    J1o = Jfx[rg1]; J2o = Jfx[rg2];
                    U1o = U[g1]; U2o = U[g2];
                    const StepRec rr = recs[ls];
                    const u64 M = (u64)(Ecur > dm.SC ? Ecur : dm.SC);
                    const u64 bh = __umul64hi(rr.thr, M), bl = rr.thr * M;
                    always = (rr.flags & 4u) || (bh >> 31);
                    bound = (bh << 32) | (bl >> 32);
                }
                i64 e1 = 0, e2 = 0;
                if (touchW) {
                    bool landed = rp_mbar_wait(mbar, phase, A.wait_polls);
                    // (once more before giving up, so that a copy still in flight has had twice the limit to land
                    // before this chain's shared memory is handed to another one)
                    if (!landed) landed = rp_mbar_wait(mbar, phase, A.wait_polls);
                    phase ^= 1u;
                    // Inspection hook: chain 0 waits once more, on a phase that nothing completes.
                    if (landed && A.stall_test && j == 0) landed = rp_mbar_wait(mbar, phase, A.wait_polls);
                    if (!__all_sync(0xffffffffu, landed)) {
                        // The bounded wait ran out: raise the status word and leave without storing anything (the
                        // level barrier and every later level then do nothing, and rp_anneal reports the time-out).
                        if (lane == 0) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
                        return;
                    }
                    rp_warp_staged_score(lane, dm.L, cpl, sum32, swap, s_qi, s_q2, s_w1, s_w2, e1, e2);
                }
                // ---- exact new score and the Metropolis decision, lane 0 ---------------------------------
                i64 n0 = 0, n1 = 0, n2 = 0, J1n = 0, J2n = 0, U1n = 0, U2n = 0;
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
                int acc_i = 0;
                if (lane == 0) {
                    const i64 en = rp_energy(n0, n1, n2);
                    const bool acc = rp_lex_less(n0, n1, n2, S0, S1, S2) || en <= Ecur || always || (u64)(en - Ecur) < bound;
                    chain->n_feas += 1;
                    if (touchW) chain->n_bytes += (i64)((swap ? 4 : 3) + (acc ? 2 : 0)) * LP * 4;
                    if (acc) {
                        chain->n_acc += 1;
                        if (touchW) {
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
                        cells[m.i] = (unsigned short)c2;
                        if (swap) cells[m.i2] = (unsigned short)c1;
                        T[c1] = (int)Ta; Q[c1] = (u64)Qa; T[c2] = (int)Tb; Q[c2] = (u64)Qb;
                        if (!swap) { cnt[c1] -= 1; cnt[c2] += 1; }
                        Esum[rg1] = e1; Afx[rg1] = A1; Jfx[rg1] = J1n;
                        if (touchW) { Esum[rg2] = e2; Afx[rg2] = A2; Jfx[rg2] = J2n; }
                        if (!ID) {
                            attkey[c1] = dm.asum * dm.C * Ta + dm.bsum * Qa; attkey[c2] = dm.asum * dm.C * Tb + dm.bsum * Qb;
                            for (int x = dpo[g1]; x < dpo[g1 + 1]; ++x) { const int c = rowbase[c1] + dpl[x]; Jcell[c] = J1n; Acell[c] = A1; }
                            for (int x = dpo[g2]; x < dpo[g2 + 1]; ++x) { const int c = rowbase[c2] + dpl[x]; Jcell[c] = J2n; Acell[c] = A2; }
                        }
                        U[g1] = U1n; U[g2] = U2n;
                        Sc[0] = n0; Sc[1] = n1; Sc[2] = n2; Sc[3] = en;
                        const u32 second = swap ? (u32)m.i2 : (u32)c2;
                        int nlog = chain->nlog;
                        if (nlog < A.log_cap) A.log[(size_t)j * A.log_cap + nlog] = make_uint2((u32)m.i, second | (swap ? 0u : 0x80000000u));
                        chain->nlog = ++nlog;
                        const u64 code = ((u64)(swap ? 0 : 1) << 63) ^ ((u64)(u32)k << 40) ^ ((u64)(u32)m.i << 20) ^ (u64)second;
                        chain->dig = (chain->dig ^ code) * 0x100000001B3ull;
                        if (rp_lex_less(n0, n1, n2, chain->B[0], chain->B[1], chain->B[2])) {
                            chain->B[0] = n0; chain->B[1] = n1; chain->B[2] = n2;
                            chain->best_step = k + 1; chain->best_nlog = nlog;
                            chain->n_imp += 1;
                        }
                    }
                    acc_i = acc ? 1 : 0;
                }
                acc_i = __shfl_sync(0xffffffffu, acc_i, 0);
                __syncwarp();                                               // lane 0's updates (slice table included) are visible
                if (acc_i) {
                    if (touchW) {
                        // the two new slices, stored where the slice table points after lane 0's update
                        int4 *o1 = (int4 *)(A.W + (size_t)wtab[rg1] * LP);
                        int4 *o2 = (int4 *)(A.W + (size_t)wtab[rg2] * LP);
                        rp_warp_staged_commit(lane, nchunks, swap, s_qi, s_q2, s_w1, s_w2, o1, o2);
                        // these stores are read again by bulk copies: order them before the asynchronous proxy
                        asm volatile("fence.proxy.async.global;" ::: "memory");
                    }
                    // the cached cells of the steps still to come follow the move
                    const bool rl = sr.flags & 1u;
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        if (x >= 2 && rl) continue;
                        if (sr.i[x] == m.i) sr.c[x] = c2;
                        else if (swap && sr.i[x] == m.i2) sr.c[x] = c1;
                    }
                    __syncwarp();               // the staged copies have been read: the next candidate may overwrite them
                    next_pos = ls + 1;
                    fmask = 0;
                }
            }
            pos = next_pos;
        }
        __syncwarp();                           // lane 0's stores to the assignment come before the next batch's reads
    }
    __syncwarp();

    // ---- epilogue: terminal state and the chain's report -----------------------------------------
    {
        char *bdst = A.blob_dst + (size_t)j * A.bl.bytes;
        const int nh = A.bl.off_cell >> 2;
        for (int x = lane; x < nh; x += 32) ((int *)bdst)[x] = ((const int *)sm)[x];
        int *td = (int *)(bdst + A.bl.off_wtab);
        for (int rg = lane; rg < dm.RG; rg += 32) td[rg] = wtab[rg];
    }
    if (lane == 0) {
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
}

// The level barrier as a launch of its own (one CTA), for chain kernels whose CTAs are single warps.
#define LEVEL_END_THREADS 512
__global__ void __launch_bounds__(LEVEL_END_THREADS)
k_level_end(const AnnealArgs A)
{
    extern __shared__ __align__(16) unsigned char smraw[];
    if (__ldcg(&A.status[RP_SW_TIMEOUT])) return;
    rp_level_end(A, threadIdx.x, LEVEL_END_THREADS, smraw, rp_le_ws_bytes(A, A.smem_bytes));
}

// Windows the warp-per-chain kernel takes: rank loads as slices of the pool, layers of whole
// 16-byte chunks (a power-of-two rank count of 4 to 128) and a chain that fits shared memory at
// least twice per SM.  Where L*P <= 512 the warp-per-candidate kernel is the alternative: it
// finishes a level sooner as long as all of its chains are resident at once (four per SM).
#define WARP_MIN_CHAINS (148 * 4)
bool rp_uses_warp_chains(const rp_ctx *c)
{
    const RpDims &dm = c->dm;
    if (!rp_uses_slices(dm)) return false;
    const bool vec = (dm.P >= 4) && (dm.P <= 128) && ((dm.P & (dm.P - 1)) == 0);
    if (!vec) return false;
    if (c->knob_chain_kernel == 1) return false;
    if (c->knob_chain_kernel != 2 && rp_uses_wpc(dm) && c->Ppop <= WARP_MIN_CHAINS) return false;
    const RpWarpLayout wl = rp_warp_layout(dm, c->bl, c->sl, dm.G == dm.D);
    return wl.bytes <= 100 * 1024;
}

template <bool ID>
static int launch_warp(rp_ctx *c, const AnnealArgs &A, const RpWarpLayout &wl)
{
    // (always the same value, above anything a launch asks for: contexts that plan different
    // windows at once on different host threads then never lower each other's limit)
    RP_CUDA(cudaFuncSetAttribute(k_anneal_warp<ID>, cudaFuncAttributeMaxDynamicSharedMemorySize, WARP_SMEM_OPTIN));
    k_anneal_warp<ID><<<c->Ppop, 32, wl.bytes, c->stream>>>(A, wl);
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

int rp_launch_anneal_warp(rp_ctx *c, AnnealArgs &A)
{
    const bool identity = (c->dm.G == c->dm.D);
    const RpWarpLayout wl = rp_warp_layout(c->dm, c->bl, c->sl, identity);
    A.smem_bytes = (unsigned)wl.bytes;
    if (identity) RP_TRY(launch_warp<true>(c, A, wl));
    else RP_TRY(launch_warp<false>(c, A, wl));
    // workspace of the barrier: cumulative weights and the replayed layout on chip where they fit
    size_t ws = 2 * std::max((size_t)c->Ppop * 8, (size_t)c->dm.N * 2);
    ws = std::min(std::max(ws, (size_t)16 * 1024), (size_t)200 * 1024);
    ws = (ws + 15) & ~(size_t)15;
    AnnealArgs B = A;
    B.smem_bytes = (unsigned)ws;
    RP_CUDA(cudaFuncSetAttribute(k_level_end, cudaFuncAttributeMaxDynamicSharedMemorySize, WARP_SMEM_OPTIN));
    k_level_end<<<1, LEVEL_END_THREADS, ws, c->stream>>>(B);
    g_rp_launches += 2;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
