// Chain kernel of the population annealing for windows with thousands of chains and slices of
// 512 < L*P <= 1024 ints (at most 256 cells): "warp per chain".
//
// A chain of Algorithm 3 is latency-bound: a step is a proposal, two dependent trips to L2 or HBM
// for the touched rank-load slices, an exact rescoring in 64-bit integers and a decision, each
// waiting for the one before.  What raises the throughput of a level is therefore the number of
// chains an SM keeps in flight, and that is set by what one chain occupies.  Here a chain is a
// single warp: the two tentative slices of a candidate (2 * L*P ints, 8 chunks of 16 bytes per
// lane and slice) are reduced as they arrive and kept nowhere (an accepted move builds them once
// more from L2 and stores them); the assignment is kept as one byte per sample; the chain's
// state arrives and leaves with plain loads and stores.  Fourteen
// chains are resident per SM (against six CTAs of 128 threads in the cooperative kernel), no
// block-wide barrier is left in the step loop, and nothing in the kernel waits on another CTA:
// the level barrier (incumbent, weights, ancestors) is a launch of its own behind it.
//
// The steps are the same as in the other two chain kernels: the random words and accept
// thresholds of the next 32 steps one step per lane; proposals and feasibility of those steps
// against the current state one step per lane; feasible candidates scored in step order by the
// whole warp; speculation redone after an acceptance.  Rank loads are slices of the pool shared
// copy-on-write with the ancestor (see AnnealArgs).
#include <algorithm>

#include "rp_level_end.cuh"

#define WARP_CHAINS_PER_SM 14            // assignment in shared memory
#define WARP_CHAINS_PER_SM_CG 16         // assignment in global memory
#define WARP_CHK 8                      // 16-byte chunks per lane and slice
#define WARP_PREFETCH 1                 // the next candidate's slices are prefetched into L2
#define WARP_PART 2                     // of which so many are in flight at once

struct CandW { MoveS m; int ti, t2, pad; };          // a feasible proposal and the lengths of the moved samples
struct ChainW {                                      // bookkeeping of the chain within this level
    i64 B[3];
    u64 dig;
    int best_step, best_nlog, nlog, pad;
    i64 n_feas, n_acc, n_imp, n_bytes;               // counters of the level
};

// Shared-memory plan of one chain: the blob's arrays up to the assignment at their blob offsets,
// then the assignment as bytes, the slice table, the static tables, and the kernel's own arrays.
struct RpWarpLayout {
    int off_cell8, off_wtab, off_static, off_keys, off_recs, off_cand, off_chain, off_spare, off_own, bytes;
};

static RpWarpLayout rp_warp_layout(const RpDims &dm, const RpBlob &bl, const RpStatic &sl, bool identity, bool cells_global)
{
    RpWarpLayout w;
    size_t o = ((size_t)bl.off_cell + 15) & ~(size_t)15;
    w.off_cell8 = (int)o;  o += cells_global ? 0 : (((size_t)dm.N + 15) & ~(size_t)15);
    w.off_wtab = (int)o;   o += ((size_t)4 * dm.RG + 15) & ~(size_t)15;
    w.off_static = (int)o; o += sl.bytes;
    w.off_keys = (int)o;   o += identity ? 0 : (size_t)3 * 8 * dm.K;
    w.off_recs = (int)o;   o += sizeof(StepRec) * SPEC;
    w.off_cand = (int)o;   o += sizeof(CandW) * SPEC;
    w.off_chain = (int)o;  o += sizeof(ChainW);
    w.off_spare = (int)o;  o += (size_t)4 * dm.RG;
    w.off_own = (int)o;    o += dm.RG;
    w.bytes = (int)((o + 15) & ~(size_t)15);
    return w;
}

// The assignment of the chain: one byte per sample in shared memory, or (CG) the 16-bit array of
// the chain's blob in global memory, read and written through L2 (more chains then fit an SM).
template <bool CG>
__device__ __forceinline__ int rp_cell_rd(const void *cells, int i)
{
    if (CG) return (int)__ldcg((const unsigned short *)cells + i);
    return (int)((const unsigned char *)cells)[i];
}
template <bool CG>
__device__ __forceinline__ void rp_cell_wr(void *cells, int i, int c)
{
    if (CG) ((unsigned short *)cells)[i] = (unsigned short)c;
    else ((unsigned char *)cells)[i] = (unsigned char)c;
}

// GuidedProposal + feasibility of one step (the rule of rp_propose, on the chain's assignment), also
// handing back the lengths of the moved samples, which the decision needs again.
template <bool CG>
__device__ __forceinline__ bool rp_propose_bytes(const RpDims &dm, const void *cell8, const int *T, const int *cnt,
                                                 const int *__restrict__ tt, const i64 *attkey, const i64 *Jcell, const i64 *Acell,
                                                 const StepRec &r, CandW &cd)
{
    const bool reloc = r.flags & 1u;
    const int ca = rp_cell_rd<CG>(cell8, r.i0), cb = rp_cell_rd<CG>(cell8, r.i1);
    const int xa = reloc ? r.i2 : rp_cell_rd<CG>(cell8, r.i2);
    const int xb = reloc ? r.i3 : rp_cell_rd<CG>(cell8, r.i3);
    const u64 Ja = (u64)Jcell[ca], Aa = (u64)Acell[ca];
    const u64 lh = __umul64hi((u64)r.bz, Ja), ll = (u64)r.bz * Ja;
    const u64 rh = Aa >> 32, rl = Aa << 32;
    const bool use_att = (lh < rh) || (lh == rh && ll < rl);
    const i64 *key = use_att ? attkey : Jcell;
    const i64 ka = key[ca], kb = key[cb], ta = key[xa], tb = key[xb];
    const bool src_b = kb > ka, dst_b = tb < ta;
    MoveS &m = cd.m;
    m.reloc = reloc;
    m.i = src_b ? r.i1 : r.i0;
    m.c1 = src_b ? cb : ca;
    m.c2 = dst_b ? xb : xa;
    m.i2 = reloc ? -1 : (dst_b ? r.i3 : r.i2);
    if (m.c1 == m.c2) return false;
    const int ti = __ldg(tt + m.i);
    cd.ti = ti; cd.t2 = 0; cd.pad = 0;
    if (reloc) return (cnt[m.c1] > 1) && (T[m.c2] + ti <= dm.C);
    const int t2 = __ldg(tt + m.i2);
    cd.t2 = t2;
    return (T[m.c1] - ti + t2 <= dm.C) && (T[m.c2] - t2 + ti <= dm.C);
}

// Half `h` of the pass over the two touched slices: this lane's chunks of W1' = W1 - d and
// W2' = W2 + d with d = q[i] - q[i2] (relocation: d = q[i]), all loads in flight before any is
// used.  COMMIT = false adds the busiest rank of every layer to p1, p2 (e1, e2 when the sums need
// 64 bits); COMMIT = true stores the two slices to o1, o2 instead.
template <bool COMMIT>
__device__ __forceinline__ void rp_warp_half(int h, int lane, int nchunks, int lpl, bool sum32, const int4 *__restrict__ qi,
                                             const int4 *__restrict__ q2, const int4 *w1, const int4 *w2, int4 *o1, int4 *o2,
                                             int &p1, int &p2, i64 &e1, i64 &e2)
{
    constexpr int H = WARP_PART;
    int4 d[H], a[H], b[H];
    // (the swap / relocation branch stays outside the loops: a branch between two loads would make
    // the second wait for the first)
    if (q2) {
        int4 o[H];
#pragma unroll
        for (int u = 0; u < H; ++u) {
            const int c = (h * H + u) * 32 + lane;
            if (h * H + u < WARP_CHK && c < nchunks) { d[u] = __ldg(qi + c); o[u] = __ldg(q2 + c); a[u] = w1[c]; b[u] = w2[c]; }
        }
#pragma unroll
        for (int u = 0; u < H; ++u) {
            const int c = (h * H + u) * 32 + lane;
            if (h * H + u < WARP_CHK && c < nchunks) { d[u].x -= o[u].x; d[u].y -= o[u].y; d[u].z -= o[u].z; d[u].w -= o[u].w; }
        }
    } else {
#pragma unroll
        for (int u = 0; u < H; ++u) {
            const int c = (h * H + u) * 32 + lane;
            if (h * H + u < WARP_CHK && c < nchunks) { d[u] = __ldg(qi + c); a[u] = w1[c]; b[u] = w2[c]; }
        }
    }
#pragma unroll
    for (int u = 0; u < H; ++u) {
        const int c = (h * H + u) * 32 + lane;
        int m1 = 0, m2 = 0;
        if (h * H + u >= WARP_CHK) continue;
        if (c < nchunks) {
            const int4 v1 = make_int4(a[u].x - d[u].x, a[u].y - d[u].y, a[u].z - d[u].z, a[u].w - d[u].w);
            const int4 v2 = make_int4(b[u].x + d[u].x, b[u].y + d[u].y, b[u].z + d[u].z, b[u].w + d[u].w);
            if (COMMIT) { o1[c] = v1; o2[c] = v2; }
            else { m1 = max4(v1); m2 = max4(v2); }
        }
        if (!COMMIT) {
            for (int o = lpl >> 1; o; o >>= 1) {          // busiest rank of the layer
                m1 = max(m1, __shfl_xor_sync(0xffffffffu, m1, o));
                m2 = max(m2, __shfl_xor_sync(0xffffffffu, m2, o));
            }
            if ((lane & (lpl - 1)) == 0 && c < nchunks) {
                if (sum32) { p1 += m1; p2 += m2; }
                else { e1 += m1; e2 += m2; }
            }
        }
    }
}

// ID: every DP slot is its own shard, so a cell is a row-shard and the per-cell proposal keys are
// the row-shard arrays of the blob themselves.
template <bool ID, bool CG>
__global__ void __launch_bounds__(32, CG ? WARP_CHAINS_PER_SM_CG : WARP_CHAINS_PER_SM)
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
    void *cell8 = CG ? (void *)(A.blob_dst + (size_t)blockIdx.x * A.bl.bytes + A.bl.off_cell) : (void *)(sm + wl.off_cell8);
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
    const int LP = dm.LP, nchunks = LP >> 2, lpl = dm.P >> 2;      // lanes that share a layer
    const bool sum32 = (i64)dm.L * dm.k * dm.C * ((dm.D + dm.G - 1) / dm.G) < (1ll << 31);

    // ---- prologue: the ancestor's terminal state --------------------------------------------
    {
        const char *bsrc = A.blob_src + (size_t)src * A.bl.bytes;
        const int nh = A.bl.off_cell >> 2;
        for (int x = lane; x < nh; x += 32) ((int *)sm)[x] = __ldg((const int *)bsrc + x);
        const unsigned short *cs = (const unsigned short *)(bsrc + A.bl.off_cell);
        const int n4 = dm.N >> 2;
        for (int x = lane; x < n4; x += 32) {
            const uint2 v = __ldg((const uint2 *)cs + x);
            if (CG) ((uint2 *)cell8)[x] = v;
            else ((u32 *)cell8)[x] = (v.x & 0xffu) | ((v.x >> 16) << 8) | ((v.y & 0xffu) << 16) | ((v.y >> 16) << 24);
        }
        for (int i = (n4 << 2) + lane; i < dm.N; i += 32) rp_cell_wr<CG>(cell8, i, (int)__ldg(cs + i));
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
        if (lane < nb) recs[lane] = rp_make_step_rec(A, A.level, A.tau, (u32)(kb + lane), (u32)j);
        __syncwarp();
        int pos = 0;
        while (pos < nb) {
            // proposals of steps kb+pos .. kb+nb-1 against the current state, one per lane
            bool ok = false;
            if (lane >= pos && lane < nb) {
                CandW cd;
                ok = rp_propose_bytes<CG>(dm, cell8, T, cnt, A.t, attkey, Jcell, Acell, recs[lane], cd);
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
                const int rg1 = rg_of[m.c1], rg2 = rg_of[m.c2];
                const bool touchW = (rg1 != rg2);
#if WARP_PREFETCH
                if (fmask) {
                    // The candidate after this one is scored if this one is rejected: start its two slices on
                    // their way from HBM to L2 now, one 128-byte line per lane and slice (no registers held).
                    const int ln = __ffs(fmask) - 1;
                    const int ra = rg_of[cand[ln].m.c1], rb = rg_of[cand[ln].m.c2];
                    if (ra != rb && lane * 32 < LP) {
                        const int *pa = A.W + (size_t)wtab[ra] * LP + lane * 32, *pb = A.W + (size_t)wtab[rb] * LP + lane * 32;
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(pa));
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(pb));
                    }
                }
#endif
                i64 e1 = 0, e2 = 0;
                const int4 *qi = (const int4 *)(A.q + (size_t)m.i * LP);
                const int4 *q2 = swap ? (const int4 *)(A.q + (size_t)m.i2 * LP) : nullptr;
                const int4 *w1 = (const int4 *)(A.W + (size_t)wtab[rg1] * LP);
                const int4 *w2 = (const int4 *)(A.W + (size_t)wtab[rg2] * LP);
                if (touchW) {
                    int p1 = 0, p2 = 0;
#pragma unroll
                    for (int h = 0; h < (WARP_CHK + WARP_PART - 1) / WARP_PART; ++h)
                        rp_warp_half<false>(h, lane, nchunks, lpl, sum32, qi, q2, w1, w2, nullptr, nullptr, p1, p2, e1, e2);
                    if (sum32) {
                        e1 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)p1);
                        e2 = (i64)__reduce_add_sync(0xffffffffu, (unsigned)p2);
                    } else {
                        e1 = warp_sum_i64(e1);
                        e2 = warp_sum_i64(e2);
                    }
                }
                // exact new score and the Metropolis decision, lane 0
                const int c1 = m.c1, c2 = m.c2;
                const int g1 = g_of[c1], g2 = g_of[c2];
                i64 n0 = 0, n1 = 0, n2 = 0, A1 = 0, A2 = 0, J1n = 0, J2n = 0, U1n = 0, U2n = 0;
                i64 Ta = 0, Qa = 0, Tb = 0, Qb = 0;
                int fb0 = 0, fb2 = 0;
                if (lane == 0) {
                    const i64 S0 = Sc[0], S1 = Sc[1], S2 = Sc[2];
                    const i64 ti = cand[ls].ti, t2 = cand[ls].t2;
                    Ta = (i64)T[c1] - ti + t2; Qa = (i64)Q[c1] - ti * ti + t2 * t2;
                    Tb = (i64)T[c2] + ti - t2; Qb = (i64)Q[c2] + ti * ti - t2 * t2;
                    if (!touchW) { e1 = Esum[rg1]; e2 = e1; }
                    const i64 aC = dm.asum * dm.C, bS = dm.bsum;
                    if (ID) { A1 = aC * Ta + bS * Qa; A2 = aC * Tb + bS * Qb; }
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
                        rp_cell_wr<CG>(cell8, m.i, c2);
                        if (swap) rp_cell_wr<CG>(cell8, m.i2, c1);
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
                        // The two slices are built once more (their sources are in L2 now) and stored
                        // where the slice table points after lane 0's update: in place or to the spares.
                        int4 *o1 = (int4 *)(A.W + (size_t)wtab[rg1] * LP);
                        int4 *o2 = (int4 *)(A.W + (size_t)wtab[rg2] * LP);
                        int p1 = 0, p2 = 0;
                        i64 x1 = 0, x2 = 0;
#pragma unroll
                        for (int h = 0; h < (WARP_CHK + WARP_PART - 1) / WARP_PART; ++h)
                            rp_warp_half<true>(h, lane, nchunks, lpl, sum32, qi, q2, w1, w2, o1, o2, p1, p2, x1, x2);
                    }
                    next_pos = ls + 1;
                    fmask = 0;
                }
            }
            pos = next_pos;
        }
    }
    __syncwarp();

    // ---- epilogue: terminal state and the chain's report -----------------------------------------
    {
        char *bdst = A.blob_dst + (size_t)j * A.bl.bytes;
        const int nh = A.bl.off_cell >> 2;
        for (int x = lane; x < nh; x += 32) ((int *)bdst)[x] = ((const int *)sm)[x];
        if (!CG) {
            unsigned short *cd = (unsigned short *)(bdst + A.bl.off_cell);
            const int n4 = dm.N >> 2;
            for (int x = lane; x < n4; x += 32) {
                const u32 v = ((const u32 *)cell8)[x];
                ((uint2 *)cd)[x] = make_uint2((v & 0xffu) | (((v >> 8) & 0xffu) << 16), ((v >> 16) & 0xffu) | ((v >> 24) << 16));
            }
            for (int i = (n4 << 2) + lane; i < dm.N; i += 32) cd[i] = (unsigned short)rp_cell_rd<false>(cell8, i);
        }
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

// Windows the warp-per-chain kernel takes: slices in the pool, 16-byte chunks of L*P <= 1024 ints
// with a power-of-two rank count, and more chains than the 128-thread kernel keeps resident (6 per
// SM; fewer chains run faster with 128 threads each).
// The assignment stays in shared memory, a byte per sample, wherever a cell fits a byte (faster:
// proposals read it four times per step); else the chain works on its blob's 16-bit array in L2.
static bool rp_warp_cells_global(const rp_ctx *c)
{
    return c->knob_chain_kernel == 3 || c->dm.K > 256;
}
bool rp_uses_warp_chains(const rp_ctx *c)
{
    const RpDims &dm = c->dm;
    if (rp_uses_wpc(dm) || !rp_uses_slices(dm) || c->knob_stall) return false;
    const bool vec = (dm.P >= 4) && (dm.P <= 128) && ((dm.P & (dm.P - 1)) == 0);
    if (!vec || dm.LP > WARP_CHK * 32 * 4) return false;
    if (c->knob_chain_kernel == 1) return false;
    if (c->knob_chain_kernel < 2 && c->Ppop <= 148 * 6) return false;
    const RpWarpLayout wl = rp_warp_layout(dm, c->bl, c->sl, dm.G == dm.D, rp_warp_cells_global(c));
    return wl.bytes <= 96 * 1024;
}

template <bool ID, bool CG>
static int launch_warp(rp_ctx *c, const AnnealArgs &A, const RpWarpLayout &wl)
{
    if (wl.bytes > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_anneal_warp<ID, CG>, cudaFuncAttributeMaxDynamicSharedMemorySize, wl.bytes));
    k_anneal_warp<ID, CG><<<c->Ppop, 32, wl.bytes, c->stream>>>(A, wl);
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

int rp_launch_anneal_warp(rp_ctx *c, AnnealArgs &A)
{
    const bool identity = (c->dm.G == c->dm.D), cg = rp_warp_cells_global(c);
    const RpWarpLayout wl = rp_warp_layout(c->dm, c->bl, c->sl, identity, cg);
    A.smem_bytes = (unsigned)wl.bytes;
    if (identity) { if (cg) RP_TRY((launch_warp<true, true>(c, A, wl))); else RP_TRY((launch_warp<true, false>(c, A, wl))); }
    else { if (cg) RP_TRY((launch_warp<false, true>(c, A, wl))); else RP_TRY((launch_warp<false, false>(c, A, wl))); }
    // workspace of the barrier: cumulative weights and the replayed layout on chip where they fit
    size_t ws = 2 * std::max((size_t)c->Ppop * 8, (size_t)c->dm.N * 2);
    ws = std::min(std::max(ws, (size_t)16 * 1024), (size_t)200 * 1024);
    ws = (ws + 15) & ~(size_t)15;
    AnnealArgs B = A;
    B.smem_bytes = (unsigned)ws;
    if (ws > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_level_end, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ws));
    k_level_end<<<1, LEVEL_END_THREADS, ws, c->stream>>>(B);
    g_rp_launches += 2;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
