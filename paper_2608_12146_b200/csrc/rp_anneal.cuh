// Shared pieces of the two chain kernels of the population annealing (Algorithm 3):
// kernel arguments, the state-independent step record, the proposal rule and the
// vectorised two-slice scoring pass.
#pragma once
#include "rp_score.cuh"

struct AnnealArgs {
    RpDims dm;
    const int *t, *q, *edp, *dp_list, *dp_off;
    const unsigned short *cell_src;  unsigned short *cell_dst;
    const int *W_src;                int *W_dst;
    const i64 *Esum_src;             i64 *Esum_dst;
    const int *anc;
    int level, steps, t_in_smem, log_cap;
    u64 tau, rho_q32, guide_q32;
    u32 key0, key1;
    i64 *term, *best;
    int *best_step, *best_nlog;
    u64 *digest;
    uint2 *log;
    i64 *counters;
    int *status;
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
__device__ __forceinline__ StepRec rp_make_step_rec(const AnnealArgs &A, u32 k, u32 j)
{
    const RpDims &dm = A.dm;
    const uint4 a = rp_philox(k, (u32)A.level, j, 0u, A.key0, A.key1);
    const uint4 b = rp_philox(k, (u32)A.level, j, 1u, A.key0, A.key1);
    const uint4 xw = rp_philox(k, (u32)A.level, j, 2u, A.key0, A.key1);
    const bool reloc = (u64)a.x < A.rho_q32, guided = (u64)a.y < A.guide_q32;
    StepRec r;
    r.i0 = rp_pick(a.z, dm.N);
    if (!guided) { r.i1 = reloc ? rp_pick(a.w, dm.K) : rp_pick(a.w, dm.N); r.i2 = 0; r.i3 = 0; }
    else {
        r.i1 = rp_pick(a.w, dm.N);
        r.i2 = reloc ? rp_pick(b.x, dm.K) : rp_pick(b.x, dm.N);
        r.i3 = reloc ? rp_pick(b.y, dm.K) : rp_pick(b.y, dm.N);
    }
    r.bz = b.z;
    const u64 nl = rp_nl2(xw.x);
    const u64 hi = __umul64hi(A.tau, nl), lo = A.tau * nl;
    const bool sat = (hi >> 30) != 0;
    r.thr = (hi << 32) | (lo >> 32);
    r.flags = (reloc ? 1u : 0u) | (guided ? 2u : 0u) | (sat ? 4u : 0u);
    return r;
}

// Tables of the chain state the proposal rule reads (all in shared memory).
struct RpChainView {
    const unsigned short *cell_of, *rg_of;
    const int *T, *cnt, *tt;
    const u64 *Q;
    const i64 *Jfx, *Afx;
};

// GuidedProposal + feasibility of one step against the current state.
//   uniform branch: sample i0, partner sample / destination cell i1.
//   guided branch: tournament of two.  Source candidates i0, i1; the comparison key is the
//   attention cost of the candidate's cell with probability Afx/Jfx of the first candidate's
//   row-shard (bz * Jfx < Afx * 2^32), else the row-shard cost Jfx; source = larger key
//   (tie: first).  Target candidates i2, i3 (samples for a swap, cells for a relocation);
//   target = smaller key (tie: first).
// Feasible = distinct cells, both cells within the token cap afterwards, no cell emptied.
__device__ __forceinline__ bool rp_propose(const RpDims &dm, const RpChainView &v, const StepRec &r,
                                           i64 aC, i64 bS, MoveS &m)
{
    const bool reloc = r.flags & 1u, guided = r.flags & 2u;
    m.reloc = reloc; m.i2 = -1;
    if (!guided) {
        m.i = r.i0;
        m.c1 = v.cell_of[m.i];
        if (reloc) m.c2 = r.i1;
        else { m.i2 = r.i1; m.c2 = v.cell_of[m.i2]; }
    } else {
        const int sa = r.i0, sb = r.i1;
        const int ca = v.cell_of[sa], cb = v.cell_of[sb];
        const int rga = v.rg_of[ca];
        const u64 Ja = (u64)v.Jfx[rga], Aa = (u64)v.Afx[rga];
        const u64 lh = __umul64hi((u64)r.bz, Ja), ll = (u64)r.bz * Ja;
        const u64 rh = Aa >> 32, rl = Aa << 32;
        const bool use_att = (lh < rh) || (lh == rh && ll < rl);
        int xa, xb, ya = -1, yb = -1;
        if (reloc) { xa = r.i2; xb = r.i3; }
        else { ya = r.i2; yb = r.i3; xa = v.cell_of[ya]; xb = v.cell_of[yb]; }
        i64 ka, kb, ta, tb;
        if (use_att) {
            ka = aC * (i64)v.T[ca] + bS * (i64)v.Q[ca];
            kb = aC * (i64)v.T[cb] + bS * (i64)v.Q[cb];
            ta = aC * (i64)v.T[xa] + bS * (i64)v.Q[xa];
            tb = aC * (i64)v.T[xb] + bS * (i64)v.Q[xb];
        } else {
            ka = (i64)Ja;
            kb = v.Jfx[v.rg_of[cb]];
            ta = v.Jfx[v.rg_of[xa]];
            tb = v.Jfx[v.rg_of[xb]];
        }
        m.i = (kb > ka) ? sb : sa;
        m.c1 = (kb > ka) ? cb : ca;
        m.c2 = (tb < ta) ? xb : xa;
        if (!reloc) m.i2 = (tb < ta) ? yb : ya;
    }
    if (m.c1 == m.c2) return false;
    const int ti = v.tt[m.i];
    if (reloc) return (v.cnt[m.c1] > 1) && (v.T[m.c2] + ti <= dm.C);
    const int t2 = v.tt[m.i2];
    return (v.T[m.c1] - ti + t2 <= dm.C) && (v.T[m.c2] - t2 + ti <= dm.C);
}

__device__ __forceinline__ int max4(const int4 &v) { return max(max(v.x, v.y), max(v.z, v.w)); }

// Tentative rank loads of the two touched row-shards, W1' = W1 - d and W2' = W2 + d with
// d = q[i] - q[i2] (relocation: d = q[i]), written to s1/s2, together with this thread's
// share of sum_l max_p W' for both.  NTH threads cooperate (tid in [0,NTH)); whole warps must
// call.  Vector form: 16-byte loads, CH chunks per thread in flight, ranks of a layer reduced
// by segmented shuffles; needs P a power of two, 4 <= P <= 128.
template <int CH, int NTH>
__device__ __forceinline__ void rp_slices_vec(int nchunks, int lanes_per_layer, const int4 *__restrict__ qi,
                                              const int4 *__restrict__ q2, const int4 *w1, const int4 *w2,
                                              int4 *s1, int4 *s2, int tid, i64 &e1, i64 &e2)
{
    const int lane = tid & 31;
    for (int base = 0; base < nchunks; base += CH * NTH) {
        int4 d[CH], a[CH], b[CH];
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            const int c = base + u * NTH + tid;
            if (c < nchunks) {
                d[u] = __ldg(qi + c);
                if (q2) { const int4 o = __ldg(q2 + c); d[u].x -= o.x; d[u].y -= o.y; d[u].z -= o.z; d[u].w -= o.w; }
                a[u] = w1[c];
                b[u] = w2[c];
            }
        }
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            const int c = base + u * NTH + tid;
            int m1 = 0, m2 = 0;
            if (c < nchunks) {
                const int4 v1 = make_int4(a[u].x - d[u].x, a[u].y - d[u].y, a[u].z - d[u].z, a[u].w - d[u].w);
                const int4 v2 = make_int4(b[u].x + d[u].x, b[u].y + d[u].y, b[u].z + d[u].z, b[u].w + d[u].w);
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
}

__device__ __forceinline__ i64 warp_max_i64(i64 v)
{
    for (int o = 16; o; o >>= 1) { i64 x = __shfl_xor_sync(0xffffffffu, v, o); v = x > v ? x : v; }
    return v;
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
__device__ __forceinline__ bool rp_mbar_wait(u64 *mbar, u32 parity)
{
    const u32 addr = rp_smem_addr(mbar);
    for (int it = 0; it < (1 << 22); ++it) {
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
