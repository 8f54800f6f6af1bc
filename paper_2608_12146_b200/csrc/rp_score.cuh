// Device routines shared by the full-evaluation kernel and the annealing kernel: the
// EDP-shard-aware objective of Sections 3.4-3.5 in integer units (score scale 2^8*C^2).
#pragma once
#include "rp_common.cuh"

// Shared-memory view of one layout's cached terms.
struct RpSmemState {
    unsigned short *cell_of;   // [N]
    int *T;                    // [K]   token sum per cell (<= C)
    u64 *Q;                    // [K]   squared-length sum per cell
    int *cnt;                  // [K]
    i64 *Esum;                 // [RG]  sum_l max_p W
    i64 *Afx;                  // [RG]  attention cost of the row-shard
    i64 *U;                    // [G]
};

__device__ __forceinline__ int rp_rowshard(const RpDims &dm, const int *__restrict__ edp, int cell)
{
    return (cell / dm.D) * dm.G + edp[cell % dm.D];
}

// Attention cost of row r on shard g (Eq. stage-aware-attention): per stage the maximum over
// the shard's DP slots of (ahat*C*T + bhat*Q) of the cell, summed over stages.  Two cells may
// be overridden with tentative statistics (c_a/c_b = -1 for none).
__device__ __forceinline__ i64 rp_attention(const RpDims &dm, const RpSmemState &st,
                                            const int *__restrict__ dp_list, const int *__restrict__ dp_off,
                                            int r, int g, int c_a, i64 Ta, i64 Qa, int c_b, i64 Tb, i64 Qb)
{
    i64 sum = 0;
    const int d0 = dp_off[g], d1 = dp_off[g + 1];
    for (int s = 0; s < dm.S; ++s) {
        i64 worst = 0;
        const i64 ca = dm.ahat[s] * dm.C, cb = dm.bhat[s];
        for (int x = d0; x < d1; ++x) {
            int c = r * dm.D + dp_list[x];
            i64 T = st.T[c], Q = (i64)st.Q[c];
            if (c == c_a) { T = Ta; Q = Qa; }
            if (c == c_b) { T = Tb; Q = Qb; }
            i64 v = ca * T + cb * Q;
            worst = v > worst ? v : worst;
        }
        sum += worst;
    }
    return sum;
}

// Warp-level "sum over layers of the maximum over ranks" of a slice whose element x = l*P+p
// is produced by f(x).  Returns the full sum in every lane.  Power-of-two P <= 32 uses
// segmented shuffles over coalesced element order; any other P walks layer by layer.
template <class F>
__device__ __forceinline__ i64 rp_warp_layer_max_sum(const RpDims &dm, int lane, F f)
{
    i64 sum = 0;
    const int P = dm.P, LP = dm.LP;
    if (P <= 32 && (P & (P - 1)) == 0) {
        for (int x0 = 0; x0 < LP; x0 += 32) {
            int x = x0 + lane;
            int v = (x < LP) ? f(x) : 0;
            for (int o = P >> 1; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
            if ((lane & (P - 1)) == 0 && x < LP) sum += v;
        }
    } else {
        for (int l = 0; l < dm.L; ++l) {
            int v = 0;
            for (int p = lane; p < P; p += 32) v = max(v, f(l * P + p));
            for (int o = 16; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
            if (lane == 0) sum += v;
        }
    }
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    return sum;
}

// Cell statistics from the assignment (Eq. cell-token-statistics), with shared-memory atomics
// (integer sums: order does not matter).  Arrays must be zeroed and the block synchronised.
__device__ __forceinline__ void rp_accumulate_cells(const RpDims &dm, const RpSmemState &st,
                                                    const int *__restrict__ t, int tid, int nt)
{
    for (int i = tid; i < dm.N; i += nt) {
        int c = st.cell_of[i];
        int ti = t[i];
        atomicAdd(&st.T[c], ti);
        atomicAdd(&st.Q[c], (u64)ti * (u64)ti);
        atomicAdd(&st.cnt[c], 1);
    }
}

// Afx for every row-shard, then U[g] and the score tuple (Eq. lexicographic-score).
// Needs Esum, T, Q in shared memory; all threads call; result valid in thread 0 after return.
__device__ __forceinline__ void rp_rows_to_score(const RpDims &dm, const RpSmemState &st,
                                                 const int *__restrict__ dp_list, const int *__restrict__ dp_off,
                                                 int tid, int nt, i64 out[3])
{
    for (int rg = tid; rg < dm.RG; rg += nt)
        st.Afx[rg] = rp_attention(dm, st, dp_list, dp_off, rg / dm.G, rg % dm.G, -1, 0, 0, -1, 0, 0);
    __syncthreads();
    for (int g = tid; g < dm.G; g += nt) {
        i64 u = 0;
        for (int r = 0; r < dm.R; ++r) u += st.Afx[r * dm.G + g] + dm.EC * st.Esum[r * dm.G + g];
        st.U[g] = u;
    }
    __syncthreads();
    if (tid == 0) {
        i64 s0 = 0, s1 = 0, s2 = 0;
        for (int g = 0; g < dm.G; ++g) { s1 += st.U[g]; s0 = st.U[g] > s0 ? st.U[g] : s0; }
        for (int rg = 0; rg < dm.RG; ++rg) {
            i64 J = st.Afx[rg] + dm.EC * st.Esum[rg];
            s2 = J > s2 ? J : s2;
        }
        out[0] = s0; out[1] = s1; out[2] = s2;
    }
}
