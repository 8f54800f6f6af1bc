// Level barrier of the population annealing (Algorithm 3): incumbent update (strictly better
// trajectory-best, lowest slot on ties) and, unless this was the last level, Boltzmann
// weights + systematic resampling -> ancestors.  Runs inside the chain kernel, in whichever
// CTA finishes last (arrival counter), so a level costs one launch.
#pragma once
#include "rp_anneal.cuh"

#define LE_MAX_WARPS 32

// Loads of values other CTAs wrote during this launch go to L2.
#define LE_LD(x) __ldcg(&(x))

// min(2^48 - 1, floor(Dd * 2^32 / M)) for 0 < M < 2^63, with rM = 2^32 / M in double precision
// (the same M for every member of a level).  The estimate Dd * rM is within one of the quotient
// (it is below 2^48 and the relative error of two roundings is below 2^-51); the exact 128-bit
// remainder then corrects it, so the result is the exact floor.  No branches: members interleave.
__device__ __forceinline__ u64 le_scaled_quotient(u64 Dd, u64 M, double rM)
{
    const bool sat = (Dd >> 16) >= M;
    u64 q = (u64)((double)Dd * rM);
    const u64 ph = __umul64hi(q, M), pl = q * M;
    const u64 nh = Dd >> 32, nl = Dd << 32;
    u64 rl = nl - pl, rh = nh - ph - (nl < pl ? 1ull : 0ull);        // remainder, signed 128-bit
#pragma unroll
    for (int it = 0; it < 2; ++it) {           // estimate too large: remainder negative
        const bool neg = (i64)rh < 0;
        const u64 t = rl + M;
        q -= neg ? 1ull : 0ull;
        rh += (neg && t < rl) ? 1ull : 0ull;
        rl = neg ? t : rl;
    }
#pragma unroll
    for (int it = 0; it < 2; ++it) {           // estimate too small: remainder at least M
        const bool big = (rh != 0) || (rl >= M);
        q += big ? 1ull : 0ull;
        rh -= (big && rl < M) ? 1ull : 0ull;
        rl -= big ? M : 0ull;
    }
    return sat ? (1ull << 48) - 1 : q;
}

// Boltzmann weights of U members at once (independent dependency chains interleave):
// w = exp2neg(min(2^40, (eq * cq) >> 16)), eq the scaled energy gap above.
template <int U>
__device__ __forceinline__ void le_weights(const i64 (&e)[U], i64 emin, u64 M, u64 cq, u64 (&w)[U])
{
    u64 z[U], acc[U];
    const double rM = 4294967296.0 / (double)M;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const u64 eq = le_scaled_quotient((u64)(e[u] - emin), M, rM);
        const u64 zh = __umul64hi(eq, cq), zl = eq * cq;
        u64 zz = (zh >> 16) ? (1ull << 40) : ((zh << 48) | (zl >> 16));
        z[u] = zz > (1ull << 40) ? (1ull << 40) : zz;
        acc[u] = 1ull << 63;
    }
    // the fraction bits in the order of rp_exp2neg; a clear bit multiplies by one (2^63 in Q63), which is exact
    // (acc * cc) >> 63 = high word of (2*acc) * cc; acc = 2^63 (nothing applied yet) gives cc itself
    if constexpr (U == 1) {          // one member per thread: a single dependent chain, unrolled (constants inline)
#pragma unroll
        for (int i = 1; i <= 24; ++i) {
            const u64 cc = ((z[0] >> (32 - i)) & 1ull) ? RP_EXP2_Q63[i - 1] : (1ull << 63);
            acc[0] = (acc[0] >> 63) ? cc : __umul64hi(acc[0] << 1, cc);
        }
    } else {
#pragma unroll 1
        for (int i = 1; i <= 24; ++i) {
            const u64 c = RP_EXP2_Q63[i - 1];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const u64 cc = ((z[u] >> (32 - i)) & 1ull) ? c : (1ull << 63);
                acc[u] = (acc[u] >> 63) ? cc : __umul64hi(acc[u] << 1, cc);
            }
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const u64 ip = z[u] >> 32;
        w[u] = ip >= 32 ? 0 : (acc[u] >> 31) >> ip;
    }
}

// Inclusive prefix sums F[j] of the weights, U consecutive members per thread and round.
template <int U>
__device__ __forceinline__ void le_prefix_weights(int P, const i64 *term, u64 cq, int tid, int nt, i64 emin, u64 M, u64 *F,
                                                  u64 *rsum, u64 *carry_s, bool have_e = false, i64 e_mine = 0)
{
    const int lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
    for (int base = 0; base < P; base += nt * U) {
        const int j0 = base + tid * U;
        i64 e[U];
        u64 w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = j0 + u;
            if (U == 1 && have_e) e[u] = (j < P) ? e_mine : emin;       // member tid's energy is still in a register
            else e[u] = (j < P) ? rp_energy(LE_LD(term[3 * (size_t)j]), LE_LD(term[3 * (size_t)j + 1]), LE_LD(term[3 * (size_t)j + 2]))
                                : emin;
        }
        le_weights<U>(e, emin, M, cq, w);
        u64 v = 0;
#pragma unroll
        for (int u = 0; u < U; ++u) { if (j0 + u >= P) w[u] = 0; v += w[u]; w[u] = v; }     // thread-local inclusive sums
        for (int o = 1; o < 32; o <<= 1) { u64 x = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += x; }
        if (lane == 31) rsum[warp] = v;
        __syncthreads();
        if (warp == 0) {
            u64 s2 = (lane < nwarps) ? rsum[lane] : 0;
            for (int o = 1; o < 32; o <<= 1) { u64 x = __shfl_up_sync(0xffffffffu, s2, o); if (lane >= o) s2 += x; }
            rsum[lane] = s2;
        }
        __syncthreads();
        const u64 upto = *carry_s + (warp ? rsum[warp - 1] : 0) + v;       // through this thread's last member
        const u64 mine = w[U - 1];
#pragma unroll
        for (int u = 0; u < U; ++u) if (j0 + u < P) F[j0 + u] = upto - mine + w[u];
        __syncthreads();
        if (tid == nt - 1) *carry_s = upto;
        __syncthreads();
    }
}

// Lane holding the lexicographically smallest (v0, v1, v2) among the lanes with j != INT_MAX
// (lowest j on ties), by reduction instructions: for each key the smallest high word, then the
// smallest low word among the lanes still in the race.  Keys are non-negative.  Returns -1 when
// no lane has a candidate.  All lanes must call.
__device__ __forceinline__ int le_lexmin_lane(i64 v0, i64 v1, i64 v2, int j)
{
    bool alive = (j != 0x7fffffff);
    const i64 key[3] = { v0, v1, v2 };
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const u32 hi = alive ? (u32)((u64)key[k] >> 32) : 0xffffffffu;
        const u32 mh = __reduce_min_sync(0xffffffffu, hi);
        alive = alive && (hi == mh);
        const u32 lo = alive ? (u32)key[k] : 0xffffffffu;
        const u32 ml = __reduce_min_sync(0xffffffffu, lo);
        alive = alive && (lo == ml);
    }
    const int mj = (int)__reduce_min_sync(0xffffffffu, alive ? (unsigned)j : 0x7fffffffu);
    const unsigned who = __ballot_sync(0xffffffffu, alive && j == mj);
    return who ? __ffs(who) - 1 : -1;
}

// Called by all threads of one CTA (nt a multiple of 32, at most 1024).  `ws` is the CTA's
// dynamic shared memory, free once the chain has been stored: the cumulative weights and the
// replayed layout live there when they fit (global memory otherwise), which keeps the
// dependent accesses of the binary search and of the replay off the L2 round trip.
__device__ __forceinline__ void rp_level_end(const AnnealArgs &A, int tid, int nt, unsigned char *ws, size_t ws_bytes)
{
    __shared__ i64 r0[LE_MAX_WARPS], r1[LE_MAX_WARPS], r2[LE_MAX_WARPS];
    __shared__ int rj[LE_MAX_WARPS], rn[LE_MAX_WARPS], ra[LE_MAX_WARPS];
    __shared__ u64 rsum[LE_MAX_WARPS];
    __shared__ int win_j, win_n, win_a, do_update;
    __shared__ i64 rmin[LE_MAX_WARPS];
    __shared__ u64 carry_s;
    const int lane = tid & 31, warp = tid >> 5, nwarps = nt >> 5;
    const int P = A.Ppop;
    const LevelOut &O = A.lo;
    const bool F_on_chip = (size_t)P * 8 <= ws_bytes / 2;
    const bool lay_on_chip = (size_t)A.dm.N * 2 <= ws_bytes / 2;
    u64 *F = F_on_chip ? (u64 *)ws : O.F;
    unsigned short *lay_s = (unsigned short *)(ws + ws_bytes / 2);

    // trace copies of the per-chain reports
    if (O.tr_term) {
        const size_t o = (size_t)A.level * P;
        for (int x = tid; x < 3 * P; x += nt) { O.tr_term[o * 3 + x] = LE_LD(A.term[x]); O.tr_best[o * 3 + x] = LE_LD(A.best[x]); }
        for (int x = tid; x < P; x += nt) { O.tr_best_step[o + x] = LE_LD(A.best_step[x]); O.tr_digest[o + x] = LE_LD(A.digest[x]); }
    }

    // ---- incumbent: lexicographic argmin of the trajectory-best scores, lowest slot first ----
    // Only chains that beat the incumbent matter; late in the schedule there are usually none.
    const i64 i0 = O.inc_score[0], i1 = O.inc_score[1], i2 = O.inc_score[2];
    i64 b0 = i0, b1 = i1, b2 = i2;
    int bj = 0x7fffffff, bn = 0, ba = 0;
    i64 emin = 0x7fffffffffffffffll;         // smallest terminal energy, for the weights further down
    i64 e_first = 0;                         // energy of member tid (all there is to weigh when P <= nt)
    const int now0 = A.w_on_chip ? A.wloc_dst[0] : 0;      // which half of the cells this level worked in (needed at the end)
#pragma unroll 2
    for (int j = tid; j < P; j += nt) {
        const i64 s0 = LE_LD(A.best[3 * (size_t)j]), s1 = LE_LD(A.best[3 * (size_t)j + 1]), s2 = LE_LD(A.best[3 * (size_t)j + 2]);
        const i64 t0 = LE_LD(A.term[3 * (size_t)j]), t1 = LE_LD(A.term[3 * (size_t)j + 1]), t2 = LE_LD(A.term[3 * (size_t)j + 2]);
        if (rp_lex_less(s0, s1, s2, b0, b1, b2)) {    // ascending j: first wins
            b0 = s0; b1 = s1; b2 = s2; bj = j;
            if (!O.cand_layout) { bn = LE_LD(A.best_nlog[j]); ba = A.anc[j]; }     // what the replay needs, fetched with the rest
        }
        const i64 e = rp_energy(t0, t1, t2);
        if (j == tid) e_first = e;
        emin = e < emin ? e : emin;
    }
    {   // warp minimum of the (non-negative) energies: smallest high word, then smallest low word among its holders
        const u32 hi = (u32)((u64)emin >> 32), mh = __reduce_min_sync(0xffffffffu, hi);
        const u32 ml = __reduce_min_sync(0xffffffffu, hi == mh ? (u32)emin : 0xffffffffu);
        emin = (i64)(((u64)mh << 32) | ml);
    }
    if (lane == 0) rmin[warp] = emin;
    if (__syncthreads_or(bj != 0x7fffffff)) {
    {
        const int src = le_lexmin_lane(b0, b1, b2, bj);         // this warp's best, handed to lane 0
        if (src >= 0) {
            b0 = __shfl_sync(0xffffffffu, b0, src); b1 = __shfl_sync(0xffffffffu, b1, src); b2 = __shfl_sync(0xffffffffu, b2, src);
            bj = __shfl_sync(0xffffffffu, bj, src); bn = __shfl_sync(0xffffffffu, bn, src); ba = __shfl_sync(0xffffffffu, ba, src);
        }
    }
    if (lane == 0) { r0[warp] = b0; r1[warp] = b1; r2[warp] = b2; rj[warp] = bj; rn[warp] = bn; ra[warp] = ba; }
    __syncthreads();
    if (warp == 0) {                                            // the same over the warps' results
        const bool has = lane < nwarps;
        b0 = has ? r0[lane] : 0; b1 = has ? r1[lane] : 0; b2 = has ? r2[lane] : 0;
        bj = has ? rj[lane] : 0x7fffffff; bn = has ? rn[lane] : 0; ba = has ? ra[lane] : 0;
        const int src = le_lexmin_lane(b0, b1, b2, bj);
        if (src >= 0) {
            b0 = __shfl_sync(0xffffffffu, b0, src); b1 = __shfl_sync(0xffffffffu, b1, src); b2 = __shfl_sync(0xffffffffu, b2, src);
            bj = __shfl_sync(0xffffffffu, bj, src); bn = __shfl_sync(0xffffffffu, bn, src); ba = __shfl_sync(0xffffffffu, ba, src);
        }
    }
    if (tid == 0) {
        win_j = bj; win_n = bn; win_a = ba;
        do_update = rp_lex_less(b0, b1, b2, i0, i1, i2);
        if (do_update) {
            O.inc_score[0] = b0; O.inc_score[1] = b1; O.inc_score[2] = b2;
            if (O.cand_layout) *O.inc_slot = bj;         // the winner stored its best layout itself
        }
    }
    __syncthreads();
    if (do_update && !O.cand_layout) {
        const int w = win_j;
        const unsigned short *cs = (const unsigned short *)(A.blob_src + (size_t)win_a * A.bl.bytes + A.bl.off_cell);
        const uint2 *lg = A.log + (size_t)w * A.log_cap;
        const int n = win_n;
        if (lay_on_chip) {
            // the log goes through the other half of the workspace when it fits (no dependent L2 round trips)
            uint2 *lg_s = (uint2 *)ws;
            const bool log_on_chip = (size_t)n * sizeof(uint2) <= ws_bytes / 2;
            for (int i = tid; i < A.dm.N; i += nt) lay_s[i] = cs[i];
            if (log_on_chip) for (int x = tid; x < n; x += nt) lg_s[x] = LE_LD(lg[x]);
            __syncthreads();
            if (tid == 0) {      // replay the accepted moves up to the trajectory-best step
                for (int x = 0; x < n; ++x) {
                    const uint2 m = log_on_chip ? lg_s[x] : LE_LD(lg[x]);
                    const int i = (int)m.x;
                    if (m.y & 0x80000000u) lay_s[i] = (unsigned short)(m.y & 0x7fffffffu);
                    else {
                        const int i2 = (int)m.y;
                        const unsigned short c = lay_s[i];
                        lay_s[i] = lay_s[i2];
                        lay_s[i2] = c;
                    }
                }
            }
            __syncthreads();
            for (int i = tid; i < A.dm.N; i += nt) O.inc_layout[i] = lay_s[i];
        } else {
            for (int i = tid; i < A.dm.N; i += nt) O.inc_layout[i] = cs[i];
            __syncthreads();
            if (tid == 0) {
                for (int x = 0; x < n; ++x) {
                    const uint2 m = LE_LD(lg[x]);
                    const int i = (int)m.x;
                    if (m.y & 0x80000000u) O.inc_layout[i] = (int)(m.y & 0x7fffffffu);
                    else {
                        const int i2 = (int)m.y;
                        const int c = O.inc_layout[i];
                        O.inc_layout[i] = O.inc_layout[i2];
                        O.inc_layout[i2] = c;
                    }
                }
            }
        }
    }
    }     // some chain beat the incumbent
    __syncthreads();
    if (O.tr_inc && tid < 3) O.tr_inc[(size_t)A.level * 3 + tid] = O.inc_score[tid];

    if (A.last) {            // the terminal states are the population as they stand
        if (O.cand_layout) {
            const int sl = *O.inc_slot;
            if (sl >= 0) {
                const unsigned short *row = O.cand_layout + (size_t)sl * A.dm.N;
                for (int i = tid; i < A.dm.N; i += nt) O.inc_layout[i] = LE_LD(row[i]);
            }
        }
        for (int m = tid; m < P; m += nt) { O.anc_out[m] = m; O.wloc_out[m] = A.wloc_dst[m]; }
        return;
    }

    // ---- resampling -------------------------------------------------------------------------
    for (int w = 0; w < nwarps; ++w) emin = rmin[w] < emin ? rmin[w] : emin;
    if (tid == 0) carry_s = 0;
    __syncthreads();
    const u64 M = (u64)(emin > A.dm.SC ? emin : A.dm.SC);
    if (P <= nt) le_prefix_weights<1>(P, A.term, A.cq, tid, nt, emin, M, F, rsum, &carry_s, true, e_first);
    else if (P <= 2 * nt) le_prefix_weights<2>(P, A.term, A.cq, tid, nt, emin, M, F, rsum, &carry_s);
    else le_prefix_weights<4>(P, A.term, A.cq, tid, nt, emin, M, F, rsum, &carry_s);
    const u64 Ftot = F[P - 1];
    const u64 u0 = (u64)(((unsigned __int128)A.resample_x * Ftot) >> 32);
    // The cell bookkeeping further down works in shared memory when 8*P ints fit: ancestors and
    // current cells are staged beyond the cumulative weights while those are still in use.
    const bool cells_on_chip = !A.w_on_chip && !A.slices && (size_t)P * 8 * sizeof(int) <= ws_bytes && F_on_chip;
    int *anc_s = (int *)ws + 6 * (size_t)P, *now_s = anc_s + P;
    if (cells_on_chip) for (int m = tid; m < P; m += nt) now_s[m] = A.wloc_dst[m];
    int depth = 0;
    while ((1 << depth) < P) ++depth;
    constexpr int SU = 4;                       // searches per thread in flight
    for (int base = 0; base < P; base += nt * SU) {
        unsigned __int128 pos[SU];
        int lo[SU], hi[SU];
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            const int m = base + u * nt + tid;
            pos[u] = (unsigned __int128)u0 + (unsigned __int128)(m < P ? m : 0) * Ftot;
            lo[u] = 0; hi[u] = (m < P) ? P - 1 : 0;      // smallest j with P*F[j] > pos (nothing to search past the end)
        }
        if ((P & (P - 1)) == 0) {       // P = 2^depth: P*F > pos  <=>  F > floor(pos / P), a 64-bit comparison
            u64 thr[SU];
#pragma unroll
            for (int u = 0; u < SU; ++u) thr[u] = (u64)(pos[u] >> depth);
            for (int it = 0; it < depth; ++it) {
#pragma unroll
                for (int u = 0; u < SU; ++u) {
                    if (lo[u] < hi[u]) {
                        const int mid = (lo[u] + hi[u]) >> 1;
                        if (F[mid] > thr[u]) hi[u] = mid; else lo[u] = mid + 1;
                    }
                }
            }
        } else {
            for (int it = 0; it < depth; ++it) {
#pragma unroll
                for (int u = 0; u < SU; ++u) {
                    if (lo[u] < hi[u]) {
                        const int mid = (lo[u] + hi[u]) >> 1;
                        if ((unsigned __int128)P * F[mid] > pos[u]) hi[u] = mid; else lo[u] = mid + 1;
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < SU; ++u) {
            const int m = base + u * nt + tid;
            if (m < P) {
                O.anc_out[m] = lo[u];
                if (cells_on_chip) anc_s[m] = lo[u];
                if (O.tr_anc) O.tr_anc[(size_t)A.level * P + m] = lo[u];
            }
        }
    }
    __syncthreads();

    // ---- W cells of the next level.  A member that is its ancestor's only child works on in the
    // ancestor's cell; children of an ancestor with several children each get a free cell and
    // copy.  Cells: 2*P of them; the ones no surviving ancestor holds are free.
    if (A.slices) return;                  // slice mode: children share their ancestor's slices, nothing to assign
    const int *now = A.wloc_dst;           // cells the terminal states of this level sit in
    if (A.w_on_chip) {      // W goes through shared memory every level anyway: alternate between the two halves
        // every member sits in the same half (its own cell m or P + m)
        for (int m = tid; m < P; m += nt) O.wloc_out[m] = (now0 >= P) ? m : P + m;
        return;
    }
    int *kids = cells_on_chip ? (int *)ws : O.scratch;     // [P]   children per ancestor
    int *need = kids + P;                  // [P]   1 = this member needs a fresh cell -> exclusive ranks
    int *isfree = need + P;                // [2P]  1 = free cell -> exclusive ranks
    int *freelist = isfree + 2 * P;        // [2P]  k-th free cell
    const int *anc_r = cells_on_chip ? anc_s : O.anc_out;
    const int *now_r = cells_on_chip ? now_s : now;
    for (int a = tid; a < P; a += nt) kids[a] = 0;
    for (int c2 = tid; c2 < 2 * P; c2 += nt) isfree[c2] = 1;
    __syncthreads();
    for (int m = tid; m < P; m += nt) atomicAdd(&kids[anc_r[m]], 1);
    __syncthreads();
    for (int a = tid; a < P; a += nt) if (kids[a] >= 1) isfree[now_r[a]] = 0;
    for (int m = tid; m < P; m += nt) need[m] = (kids[anc_r[m]] != 1);
    __syncthreads();
    // exclusive prefix sums of need[P] and isfree[2P]: a thread scans its own consecutive chunk, one
    // block-wide scan of the chunk totals joins them
    for (int pass = 0; pass < 2; ++pass) {
        int *arr = pass ? isfree : need;
        const int n = pass ? 2 * P : P;
        const int chunk = (n + nt - 1) / nt;
        const int x0 = min(n, tid * chunk), x1 = min(n, x0 + chunk);
        int total = 0;
        for (int x = x0; x < x1; ++x) total += arr[x];
        int v = total;
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += y; }
        if (lane == 31) rj[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int s2 = (lane < nwarps) ? rj[lane] : 0;
            for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, s2, o); if (lane >= o) s2 += y; }
            rj[lane] = s2;
        }
        __syncthreads();
        int rank = (warp ? rj[warp - 1] : 0) + v - total;          // exclusive rank of the chunk's first element
        for (int x = x0; x < x1; ++x) {
            const int flag = arr[x];
            if (pass) { if (flag) freelist[rank] = x; }
            else arr[x] = flag ? rank : -1;
            rank += flag;
        }
        __syncthreads();
    }
    for (int m = tid; m < P; m += nt)
        O.wloc_out[m] = (need[m] >= 0) ? freelist[need[m]] : now_r[anc_r[m]];
}

// Shared-memory bytes the level barrier works in: all of the CTA's dynamic shared memory, unless
// the inspection hook caps it (which sends the cumulative weights, the replayed layout and the
// cell bookkeeping through their global-memory forms on windows of any size).
__device__ __forceinline__ size_t rp_le_ws_bytes(const AnnealArgs &A, size_t ws_bytes)
{
    return (A.le_ws_cap && A.le_ws_cap < ws_bytes) ? (size_t)A.le_ws_cap : ws_bytes;
}

// Tail of a chain CTA: publish, take a ticket, and let the last arrival run the level barrier.
__device__ __forceinline__ void rp_finish_level(const AnnealArgs &A, int tid, int nt, unsigned char *ws, size_t ws_bytes)
{
    __shared__ int is_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(A.lo.done, 1);
        is_last = (ticket == (int)gridDim.x - 1);
        if (is_last) {
            *A.lo.done = 0;
            if (__ldcg(&A.status[RP_SW_TIMEOUT])) is_last = 0;              // some chain gave up: no barrier, the call fails
        }
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    rp_level_end(A, tid, nt, ws, rp_le_ws_bytes(A, ws_bytes));
}
