// Chain kernel of the population annealing for latency-bound windows (L*P <= 512):
// "warp per candidate".
//
// One CTA of NW warps runs one chain.  The random words and accept thresholds of the next
// NW*32 steps are computed one step per thread.  The leading warp then evaluates the
// proposals of the next 32 steps against the current state, one step per lane (a proposal
// depends on the state, and the state changes only when a move is accepted).  The feasible
// ones are scored NW at a time, one candidate per warp, all against the same state: each
// warp builds the two tentative rank-load slices with 16-byte loads, reduces the busiest
// rank per layer with shuffles, rebuilds the exact score and takes the Metropolis decision.
// The first accepted candidate in step order is committed by its warp and everything
// speculated after it is discarded and redone; if none is accepted the next NW follow.
// This is step-for-step the sequential chain of Algorithm 3: a later step is only ever
// scored against the state it would have seen.
//
// The rank-load tensor W of the chain sits in shared memory when it fits (moved in and out
// with bulk asynchronous copies), so a scoring pass reads only the moved samples' demand
// rows from L2.
#include "rp_anneal.cuh"

struct EvalRes {
    int acc, touchW, rg1, rg2, g1, g2, pad0, pad1;
    i64 e1, e2, A1, A2, J1n, J2n, U1n, U2n, n0, n1, n2, en, Ta, Qa, Tb, Qb, bytes;
};
struct ChainS {
    i64 S[3], Ecur, B[3];
    u64 dig;
    i64 n_feas, n_acc, n_imp, n_bytes;
    int best_step, best_nlog, nlog, failed;
};

template <int NW, bool WS, int CH>
__global__ void __launch_bounds__(NW * 32)
k_anneal_wpc(const AnnealArgs A)
{
    constexpr int NT = NW * 32;
    const RpDims &dm = A.dm;
    extern __shared__ __align__(16) unsigned char smraw[];
    u64 *Q = (u64 *)smraw;
    i64 *Esum = (i64 *)(Q + dm.K);
    i64 *Afx = Esum + dm.RG;
    i64 *Jfx = Afx + dm.RG;
    i64 *U = Jfx + dm.RG;
    StepRec *recs = (StepRec *)(U + dm.G);
    EvalRes *res = (EvalRes *)(recs + NT);
    ChainS *chain = (ChainS *)(res + NW);
    u64 *mbar = (u64 *)(chain + 1);
    int *scratch = (int *)(((uintptr_t)(mbar + 1) + 15) & ~(uintptr_t)15);
    const size_t wn = (size_t)dm.RG * dm.LP;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;           // keeps every slice 16-byte aligned
    int *Wsm = scratch + (size_t)NW * 2 * slice_pad;
    int *T = Wsm + (WS ? ((wn + 3) & ~(size_t)3) : 0);
    int *cnt = T + dm.K;
    int *dpl = cnt + dm.K;
    int *dpo = dpl + dm.D;
    MoveS *mvs = (MoveS *)(dpo + dm.G + 1);
    int *rnd = (int *)(mvs + SPEC);                                     // [0] feasible mask
    int *t_s = rnd + 2;
    unsigned short *cell_of = (unsigned short *)(t_s + (A.t_in_smem ? dm.N : 0));
    unsigned short *rg_of = cell_of + dm.N;
    unsigned short *g_of = rg_of + dm.K;
    unsigned short *rowbase = g_of + dm.K;
    RpSmemState st = { cell_of, T, Q, cnt, Esum, Afx, U };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int j = blockIdx.x;
    const int src = A.anc[j];
    const int *tt = A.t_in_smem ? t_s : A.t;
    const bool identity_edp = (dm.G == dm.D);
    int *Wj = WS ? Wsm : A.W_dst + (size_t)j * wn;
    const bool bulk_ok = WS && ((wn & 3) == 0);
    const bool vec = (dm.P >= 4) && (dm.P <= 128) && ((dm.P & (dm.P - 1)) == 0);
    const i64 aC = dm.asum * dm.C, bS = dm.bsum;

    // ---- prologue: adopt the ancestor's terminal state -------------------------------
    {
        const int *ws = A.W_src + (size_t)src * wn;
        if (tid == 0) chain->failed = 0;
        if (bulk_ok) {
            if (tid == 0) {
                rp_mbar_init(mbar, 1);
                rp_mbar_expect_tx(mbar, (u32)(wn * 4));
                for (size_t off = 0; off < wn * 4; off += 32768) {
                    const u32 n = (u32)((wn * 4 - off) < 32768 ? (wn * 4 - off) : 32768);
                    rp_bulk_g2s((char *)Wsm + off, (const char *)ws + off, n, mbar);
                }
            }
        } else if ((wn & 3) == 0) {
            const int4 *ws4 = (const int4 *)ws;
            int4 *wd4 = (int4 *)Wj;
#pragma unroll 8
            for (size_t x = tid; x < wn / 4; x += NT) wd4[x] = ws4[x];
        } else {
            for (size_t x = tid; x < wn; x += NT) Wj[x] = ws[x];
        }
        const unsigned short *cs = A.cell_src + (size_t)src * dm.N;
        for (int i = tid; i < dm.N; i += NT) cell_of[i] = cs[i];
        if (A.t_in_smem) for (int i = tid; i < dm.N; i += NT) t_s[i] = A.t[i];
        for (int c = tid; c < dm.K; c += NT) {
            T[c] = 0; Q[c] = 0; cnt[c] = 0;
            const int r = c / dm.D, g = A.edp[c % dm.D];
            rg_of[c] = (unsigned short)(r * dm.G + g);
            g_of[c] = (unsigned short)g;
            rowbase[c] = (unsigned short)(r * dm.D);
        }
        for (int d = tid; d < dm.D; d += NT) dpl[d] = A.dp_list[d];
        for (int g = tid; g <= dm.G; g += NT) dpo[g] = A.dp_off[g];
        const i64 *es = A.Esum_src + (size_t)src * dm.RG;
        for (int rg = tid; rg < dm.RG; rg += NT) Esum[rg] = es[rg];
    }
    __syncthreads();
    rp_accumulate_cells(dm, st, tt, tid, NT);
    __syncthreads();
    {
        i64 S[3];
        rp_rows_to_score(dm, st, dpl, dpo, tid, NT, S);
        for (int rg = tid; rg < dm.RG; rg += NT) Jfx[rg] = Afx[rg] + dm.EC * Esum[rg];
        if (tid == 0) {
            chain->S[0] = S[0]; chain->S[1] = S[1]; chain->S[2] = S[2];
            chain->B[0] = S[0]; chain->B[1] = S[1]; chain->B[2] = S[2];
            chain->Ecur = rp_energy(S[0], S[1], S[2]);
            chain->dig = 0; chain->n_feas = 0; chain->n_acc = 0; chain->n_imp = 0; chain->n_bytes = 0;
            chain->best_step = 0; chain->best_nlog = 0; chain->nlog = 0;
        }
    }
    bool copy_ok = true;
    if (bulk_ok) copy_ok = rp_mbar_wait(mbar, 0);
    if (!copy_ok) chain->failed = 1;
    __syncthreads();
    if (chain->failed) {                 // the bulk copy never landed: report and leave
        if (tid == 0) atomicExch(&A.status[RP_SW_TIMEOUT], 1);
        return;
    }

    uint2 *logj = A.log + (size_t)j * A.log_cap;
    const RpChainView view = { cell_of, rg_of, T, cnt, tt, Q, Jfx, Afx };
    int *my_s1 = scratch + (size_t)warp * 2 * slice_pad, *my_s2 = my_s1 + slice_pad;

    for (int kb = 0; kb < A.steps; kb += NT) {
        const int nb = min(NT, A.steps - kb);
        if (tid < nb) recs[tid] = rp_make_step_rec(A, (u32)(kb + tid), (u32)j);
        __syncthreads();

        int pos = 0;
        while (pos < nb) {
            // ---- proposals of steps kb+pos .. kb+pos+31 against the current state ----
            if (warp == 0) {
                bool ok = false;
                if (pos + lane < nb) {
                    MoveS m;
                    ok = rp_propose(dm, view, recs[pos + lane], aC, bS, m);
                    if (ok) mvs[lane] = m;
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
                if (my >= 0) {
                    const MoveS m = mvs[my];
                    const bool swap = !m.reloc;
                    const int rg1 = rg_of[m.c1], rg2 = rg_of[m.c2];
                    const bool touchW = (rg1 != rg2);
                    i64 e1 = 0, e2 = 0;
                    if (touchW) {
                        const int *qi = A.q + (size_t)m.i * dm.LP;
                        const int *q2 = swap ? A.q + (size_t)m.i2 * dm.LP : nullptr;
                        const int *w1 = Wj + (size_t)rg1 * dm.LP, *w2 = Wj + (size_t)rg2 * dm.LP;
                        if (vec) {
                            rp_slices_vec<CH, 32>(dm.LP >> 2, dm.P >> 2, (const int4 *)qi, (const int4 *)q2, (const int4 *)w1,
                                                  (const int4 *)w2, (int4 *)my_s1, (int4 *)my_s2, lane, e1, e2);
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
                        e1 = warp_sum_i64(e1);
                        e2 = warp_sum_i64(e2);
                    }
                    // exact new score and the Metropolis decision
                    const int c1 = m.c1, c2 = m.c2;
                    const int g1 = g_of[c1], g2 = g_of[c2];
                    EvalRes R;
                    int fb0 = 0, fb2 = 0;
                    i64 n0 = 0, n2 = 0;
                    if (lane == 0) {
                        const i64 S0 = chain->S[0], S1 = chain->S[1], S2 = chain->S[2];
                        const i64 ti = tt[m.i], t2 = swap ? tt[m.i2] : 0;
                        R.Ta = (i64)T[c1] - ti + t2; R.Qa = (i64)Q[c1] - ti * ti + t2 * t2;
                        R.Tb = (i64)T[c2] + ti - t2; R.Qb = (i64)Q[c2] + ti * ti - t2 * t2;
                        if (!touchW) { e1 = Esum[rg1]; e2 = e1; }
                        if (identity_edp) { R.A1 = aC * R.Ta + bS * R.Qa; R.A2 = aC * R.Tb + bS * R.Qb; }
                        else {
                            R.A1 = rp_attention(dm, st, dpl, dpo, rowbase[c1] / dm.D, g1, c1, R.Ta, R.Qa, c2, R.Tb, R.Qb);
                            R.A2 = touchW ? rp_attention(dm, st, dpl, dpo, rowbase[c2] / dm.D, g2, c1, R.Ta, R.Qa, c2, R.Tb, R.Qb) : R.A1;
                        }
                        const i64 J1o = Jfx[rg1], J2o = Jfx[rg2];
                        R.J1n = R.A1 + dm.EC * e1; R.J2n = touchW ? R.A2 + dm.EC * e2 : R.J1n;
                        const i64 dJ1 = R.J1n - J1o, dJ2 = touchW ? R.J2n - J2o : 0;
                        const i64 U1o = U[g1], U2o = U[g2];
                        if (g1 == g2) { R.U1n = U1o + dJ1 + dJ2; R.U2n = R.U1n; }
                        else { R.U1n = U1o + dJ1; R.U2n = U2o + dJ2; }
                        R.n1 = S1 + dJ1 + dJ2;
                        {
                            const i64 newmax = R.U1n > R.U2n ? R.U1n : R.U2n, oldmax = U1o > U2o ? U1o : U2o;
                            if (newmax >= S0) n0 = newmax;
                            else if (oldmax < S0) n0 = S0;
                            else { n0 = newmax; fb0 = 1; }
                        }
                        {
                            const i64 newmax = R.J1n > R.J2n ? R.J1n : R.J2n, oldmax = J1o > J2o ? J1o : J2o;
                            if (newmax >= S2) n2 = newmax;
                            else if (oldmax < S2) n2 = S2;
                            else { n2 = newmax; fb2 = 1; }
                        }
                    }
                    const int fb = __shfl_sync(0xffffffffu, fb0 | (fb2 << 1), 0);
                    if (fb & 1) {       // the previous maximum sat on a changed entry and fell: rescan
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
                        const StepRec rr = recs[pos + my];
                        const i64 Ecur = chain->Ecur;
                        bool acc = rp_lex_less(n0, R.n1, n2, chain->S[0], chain->S[1], chain->S[2]);
                        const i64 en = rp_energy(n0, R.n1, n2);
                        if (!acc) {
                            if (en <= Ecur || (rr.flags & 4u)) acc = true;
                            else {
                                const u64 M = (u64)(Ecur > dm.SC ? Ecur : dm.SC);
                                const u64 bh = __umul64hi(rr.thr, M), bl = rr.thr * M;
                                acc = (bh >> 31) ? true : ((u64)(en - Ecur) < ((bh << 32) | (bl >> 32)));
                            }
                        }
                        R.acc = acc; R.touchW = touchW; R.rg1 = rg1; R.rg2 = rg2; R.g1 = g1; R.g2 = g2;
                        R.e1 = e1; R.e2 = e2; R.n0 = n0; R.n2 = n2; R.en = en;
                        R.bytes = touchW ? (i64)((swap ? 4 : 3) + (acc ? 2 : 0)) * dm.LP * 4 : 0;
                        res[warp] = R;
                    }
                }
                __syncthreads();
                const int wave = min(NW, __popc(fmask));
                int win = -1;
                for (int w = 0; w < wave; ++w) if (res[w].acc) { win = w; break; }
                if (win >= 0) {
                    if (warp == win) {
                        const MoveS m = mvs[my];
                        const EvalRes &R = res[win];
                        const bool swap = !m.reloc;
                        if (R.touchW) {
                            int *w1 = Wj + (size_t)R.rg1 * dm.LP, *w2 = Wj + (size_t)R.rg2 * dm.LP;
                            if (vec) {
                                for (int c = lane; c < (dm.LP >> 2); c += 32) {
                                    ((int4 *)w1)[c] = ((const int4 *)my_s1)[c];
                                    ((int4 *)w2)[c] = ((const int4 *)my_s2)[c];
                                }
                            } else {
                                for (int x = lane; x < dm.LP; x += 32) { w1[x] = my_s1[x]; w2[x] = my_s2[x]; }
                            }
                        }
                        if (lane == 0) {
                            const int c1 = m.c1, c2 = m.c2;
                            const int k = kb + pos + my;
                            cell_of[m.i] = (unsigned short)c2;
                            if (swap) cell_of[m.i2] = (unsigned short)c1;
                            T[c1] = (int)R.Ta; Q[c1] = (u64)R.Qa; T[c2] = (int)R.Tb; Q[c2] = (u64)R.Qb;
                            if (!swap) { cnt[c1] -= 1; cnt[c2] += 1; }
                            Esum[R.rg1] = R.e1; Afx[R.rg1] = R.A1; Jfx[R.rg1] = R.J1n;
                            if (R.touchW) { Esum[R.rg2] = R.e2; Afx[R.rg2] = R.A2; Jfx[R.rg2] = R.J2n; }
                            U[R.g1] = R.U1n; U[R.g2] = R.U2n;
                            chain->S[0] = R.n0; chain->S[1] = R.n1; chain->S[2] = R.n2; chain->Ecur = R.en;
                            const u32 second = swap ? (u32)m.i2 : (u32)c2;
                            int nlog = chain->nlog;
                            if (nlog < A.log_cap) logj[nlog] = make_uint2((u32)m.i, second | (swap ? 0u : 0x80000000u));
                            chain->nlog = ++nlog;
                            const u64 code = ((u64)(swap ? 0 : 1) << 63) ^ ((u64)(u32)k << 40) ^ ((u64)(u32)m.i << 20) ^ (u64)second;
                            chain->dig = (chain->dig ^ code) * 0x100000001B3ull;
                            if (rp_lex_less(R.n0, R.n1, R.n2, chain->B[0], chain->B[1], chain->B[2])) {
                                chain->B[0] = R.n0; chain->B[1] = R.n1; chain->B[2] = R.n2;
                                chain->best_step = k + 1; chain->best_nlog = nlog;
                                chain->n_imp += 1;
                            }
                            i64 by = 0;
                            for (int w = 0; w <= win; ++w) by += res[w].bytes;
                            chain->n_feas += win + 1; chain->n_acc += 1; chain->n_bytes += by;
                        }
                        next_pos = pos + my + 1;      // warp-local; published below
                        if (lane == 0) rnd[1] = next_pos;
                    }
                    fmask = 0;
                } else {
                    if (tid == 0) {
                        i64 by = 0;
                        for (int w = 0; w < wave; ++w) by += res[w].bytes;
                        chain->n_feas += wave; chain->n_bytes += by;
                    }
                    for (int w = 0; w < wave; ++w) fmask &= fmask - 1;
                }
                __syncthreads();
                if (win >= 0) next_pos = rnd[1];
            }
            pos = next_pos;
        }
    }

    // ---- epilogue: terminal state and chain report ------------------------------------------
    {
        unsigned short *cd = A.cell_dst + (size_t)j * dm.N;
        for (int i = tid; i < dm.N; i += NT) cd[i] = cell_of[i];
        i64 *ed = A.Esum_dst + (size_t)j * dm.RG;
        for (int rg = tid; rg < dm.RG; rg += NT) ed[rg] = Esum[rg];
        if (WS) {
            int *wd = A.W_dst + (size_t)j * wn;
            if (bulk_ok) {
                rp_fence_async_smem();
                __syncthreads();
                if (tid == 0) {
                    for (size_t off = 0; off < wn * 4; off += 32768) {
                        const u32 n = (u32)((wn * 4 - off) < 32768 ? (wn * 4 - off) : 32768);
                        rp_bulk_s2g((char *)wd + off, (const char *)Wsm + off, n);
                    }
                    rp_bulk_commit_wait();
                }
            } else {
                for (size_t x = tid; x < wn; x += NT) wd[x] = Wsm[x];
            }
        }
        if (tid == 0) {
            for (int x = 0; x < 3; ++x) { A.term[3 * (size_t)j + x] = chain->S[x]; A.best[3 * (size_t)j + x] = chain->B[x]; }
            A.best_step[j] = chain->best_step;
            A.best_nlog[j] = chain->best_nlog;
            A.digest[j] = chain->dig;
            atomicAdd((u64 *)&A.counters[0], (u64)A.steps);
            atomicAdd((u64 *)&A.counters[1], (u64)chain->n_feas);
            atomicAdd((u64 *)&A.counters[2], (u64)chain->n_acc);
            atomicAdd((u64 *)&A.counters[3], (u64)chain->n_imp);
            atomicAdd((u64 *)&A.counters[4], (u64)chain->n_bytes);
            if (src != j) atomicAdd((u64 *)&A.counters[5], (u64)2 * dm.RG * dm.LP * 4);
        }
    }
}

#define WPC_WARPS 4

// Shared-memory bytes of the warp-per-candidate kernel; *w_in_smem says whether W fits on chip
// beside a second CTA.
size_t rp_wpc_smem_bytes(const RpDims &dm, int t_in_smem, int *w_in_smem)
{
    const int NT = WPC_WARPS * 32;
    size_t b = sizeof(u64) * dm.K + sizeof(i64) * (3 * (size_t)dm.RG + dm.G) + sizeof(StepRec) * NT +
               sizeof(EvalRes) * WPC_WARPS + sizeof(ChainS) + sizeof(u64) + 16;
    const size_t slice_pad = ((size_t)dm.LP + 3) & ~(size_t)3;
    b += sizeof(int) * WPC_WARPS * 2 * slice_pad;
    size_t small = sizeof(int) * (2 * (size_t)dm.K + dm.D + dm.G + 1 + 2 + (t_in_smem ? dm.N : 0)) + sizeof(MoveS) * SPEC;
    small += sizeof(unsigned short) * ((size_t)dm.N + 3 * (size_t)dm.K) + 16;
    b += small;
    const size_t wbytes = sizeof(int) * ((((size_t)dm.RG * dm.LP) + 3) & ~(size_t)3);
    *w_in_smem = (b + wbytes <= 110 * 1024);
    if (*w_in_smem) b += wbytes;
    return (b + 15) & ~(size_t)15;
}

int rp_launch_anneal_wpc(rp_ctx *c, const AnnealArgs &A0)
{
    AnnealArgs A = A0;
    const RpDims &dm = c->dm;
    A.t_in_smem = dm.N <= 2048;
    int ws = 0;
    const size_t smem = rp_wpc_smem_bytes(dm, A.t_in_smem, &ws);
    if (smem > 220 * 1024) return RP_ERR_RANGE;
    const int chunks = ((dm.LP >> 2) + 31) / 32;
#define LAUNCH(WS_, CH_)                                                                              \
    do {                                                                                              \
        if (smem > 48 * 1024)                                                                         \
            RP_CUDA(cudaFuncSetAttribute(k_anneal_wpc<WPC_WARPS, WS_, CH_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
        k_anneal_wpc<WPC_WARPS, WS_, CH_><<<c->Ppop, WPC_WARPS * 32, smem, c->stream>>>(A);           \
    } while (0)
    if (ws) { if (chunks <= 1) LAUNCH(true, 1); else if (chunks <= 2) LAUNCH(true, 2); else LAUNCH(true, 4); }
    else { if (chunks <= 1) LAUNCH(false, 1); else if (chunks <= 2) LAUNCH(false, 2); else LAUNCH(false, 4); }
#undef LAUNCH
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
