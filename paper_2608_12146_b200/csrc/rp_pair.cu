// EDPAwarePair (Section 4.1.1; Algorithm 2, third construction operator): every completed cell
// stays the same set of samples, only the (row, DP slot) it occupies changes.
//
//   profile of cell b      w_b[l][p] = sum of q[i][l][p] over its samples; peak_b = max w_b
//   order                  cells by decreasing peak, ties by lower cell index
//   insertion key of an empty slot s (row r, shard g) for the cell in hand:
//                          (sum_l max_p (V+w_b) - sum_l max_p V,  max_{l,p} (V+w_b)),
//                          V the rank load of row-shard (r, g) from the cells placed so far;
//                          slots ranked by ascending key, ties by lower slot index
//   rank-decaying sampling rho = min(min(w, #empty) - 1, leading zero bits of the draw),
//                          draw = Philox(h, 0, member, 6).x for the h-th cell placed
//
// One CTA per population member (member 0, the length-only seed, is left alone).  Empty slots of
// one row-shard share their key, so the key is computed once per row-shard that still has an
// empty slot, one warp per row-shard, lanes over layers.
#include "rp_common.cuh"

#define PAIR_THREADS 256
#define PAIR_WARPS (PAIR_THREADS / 32)

struct PairKey { i64 d; int p; int s; };

__device__ __forceinline__ bool pair_less(const PairKey &a, const PairKey &b)
{
    if (a.d != b.d) return a.d < b.d;
    if (a.p != b.p) return a.p < b.p;
    return a.s < b.s;
}

__global__ void __launch_bounds__(PAIR_THREADS)
k_edp_pair(RpDims dm, const int *__restrict__ q, const unsigned short *__restrict__ rg_of,
           const int *__restrict__ lay_in, int *__restrict__ lay_out, int *__restrict__ prof_all,
           int *__restrict__ V_all, int first_member, int width, u32 key0, u32 key1)
{
    extern __shared__ __align__(16) unsigned char pair_smem[];
    const int N = dm.N, K = dm.K, RG = dm.RG, LP = dm.LP, L = dm.L, P = dm.P;
    i64 *e_old = (i64 *)pair_smem;                 // [RG] sum_l max_p V
    i64 *kd = e_old + RG;                          // [RG] increase of that sum for the cell in hand
    int *kp = (int *)(kd + RG);                    // [RG] largest peak after insertion
    int *free_rg = kp + RG;                        // [RG] empty slots left in the row-shard
    int *peak = free_rg + RG;                      // [K]
    int *order = peak + K;                         // [K] cells by (-peak, index)
    int *slot_of = order + K;                      // [K]
    int *cstart = slot_of + K;                     // [K + 1] first entry of each cell in `list`
    int *fillp = cstart + K + 1;                   // [K] fill pointers / empty flags later
    int *list = fillp + K;                         // [N] samples grouped by cell
    i64 *eself = (i64 *)(((size_t)(list + N) + 7) & ~(size_t)7);   // [K] sum_l max_p of the cell's own profile
    __shared__ PairKey red[PAIR_WARPS];
    __shared__ int picked[32];
    __shared__ int rho_s, chosen_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int j = first_member + blockIdx.x;
    const int *lay = lay_in + (size_t)j * N;
    int *prof = prof_all + (size_t)blockIdx.x * K * LP;
    int *V = V_all + (size_t)j * RG * LP;

    // ---- samples grouped by cell (counting sort) ----------------------------------------------
    for (int b = tid; b <= K; b += PAIR_THREADS) cstart[b] = 0;
    for (int x = tid; x < RG; x += PAIR_THREADS) { e_old[x] = 0; free_rg[x] = 0; }
    __syncthreads();
    for (int i = tid; i < N; i += PAIR_THREADS) atomicAdd(&cstart[lay[i] + 1], 1);
    for (int s = tid; s < K; s += PAIR_THREADS) atomicAdd(&free_rg[rg_of[s]], 1);
    __syncthreads();
    if (tid == 0) for (int b = 0; b < K; ++b) cstart[b + 1] += cstart[b];
    __syncthreads();
    for (int b = tid; b < K; b += PAIR_THREADS) fillp[b] = cstart[b];
    __syncthreads();
    for (int i = tid; i < N; i += PAIR_THREADS) list[atomicAdd(&fillp[lay[i]], 1)] = i;
    for (size_t x = tid; x < (size_t)RG * LP; x += PAIR_THREADS) V[x] = 0;
    __syncthreads();

    // ---- cell profiles and peaks: one warp per cell, lanes over (layer, rank) -------------------
    for (int b = warp; b < K; b += PAIR_WARPS) {
        int pk = 0;
        for (int x = lane; x < LP; x += 32) {
            int acc = 0;
            for (int e = cstart[b]; e < cstart[b + 1]; ++e) acc += __ldg(q + (size_t)list[e] * LP + x);
            prof[(size_t)b * LP + x] = acc;
            pk = max(pk, acc);
        }
        pk = __reduce_max_sync(0xffffffffu, pk);
        __syncwarp();                              // the profile row is complete before it is read back per layer
        i64 es = 0;
        for (int l = lane; l < L; l += 32) {
            int mn = 0;
            for (int p = 0; p < P; ++p) mn = max(mn, prof[(size_t)b * LP + l * P + p]);
            es += mn;
        }
        for (int o = 16; o; o >>= 1) es += __shfl_xor_sync(0xffffffffu, es, o);
        if (lane == 0) { peak[b] = pk; eself[b] = es; }
    }
    __syncthreads();
    // ---- order by (-peak, index): rank by counting ---------------------------------------------
    for (int b = tid; b < K; b += PAIR_THREADS) {
        const int pb = peak[b];
        int r = 0;
        for (int o = 0; o < K; ++o) { const int po = peak[o]; r += (po > pb) || (po == pb && o < b); }
        order[r] = b;
        fillp[b] = 1;                              // from here on: 1 = slot b is empty
    }
    __syncthreads();

    // ---- place the cells one by one ------------------------------------------------------------
    for (int h = 0; h < K; ++h) {
        const int b = order[h];
        const int *wb = prof + (size_t)b * LP;
        // keys of the row-shards that still have an empty slot
        for (int rg = warp; rg < RG; rg += PAIR_WARPS) {
            if (free_rg[rg] == 0) continue;
            if (e_old[rg] == 0) {                  // nothing placed there yet (or only empty profiles): the cell's own sums
                if (lane == 0) { kd[rg] = eself[b]; kp[rg] = peak[b]; }
                continue;
            }
            const int *v = V + (size_t)rg * LP;
            i64 en = 0;
            int pk = 0;
            for (int l = lane; l < L; l += 32) {
                int mn = 0;
                for (int p = 0; p < P; ++p) mn = max(mn, v[l * P + p] + wb[l * P + p]);
                en += mn;
                pk = max(pk, mn);
            }
            for (int o = 16; o; o >>= 1) en += __shfl_xor_sync(0xffffffffu, en, o);
            pk = __reduce_max_sync(0xffffffffu, pk);
            if (lane == 0) { kd[rg] = en - e_old[rg]; kp[rg] = pk; }
        }
        if (tid == 0) {
            const uint4 xw = rp_philox((u32)h, 0u, (u32)j, 6u, key0, key1);
            const int ne = K - h, m = ne < width ? ne : width;
            const int lz = __clz((int)xw.x);
            rho_s = lz < m - 1 ? lz : m - 1;
        }
        __syncthreads();
        // the rho-th ranked empty slot: rho + 1 rounds of a block-wide argmin, earlier picks excluded
        const int rho = rho_s;
        for (int round = 0; round <= rho; ++round) {
            PairKey best = { 0x7fffffffffffffffll, 0x7fffffff, 0x7fffffff };
            for (int s = tid; s < K; s += PAIR_THREADS) {
                if (!fillp[s]) continue;
                bool taken = false;
                for (int x = 0; x < round; ++x) taken |= (picked[x] == s);
                if (taken) continue;
                const int rg = rg_of[s];
                const PairKey k = { kd[rg], kp[rg], s };
                if (pair_less(k, best)) best = k;
            }
            for (int o = 16; o; o >>= 1) {
                PairKey ot;
                ot.d = __shfl_xor_sync(0xffffffffu, best.d, o);
                ot.p = __shfl_xor_sync(0xffffffffu, best.p, o);
                ot.s = __shfl_xor_sync(0xffffffffu, best.s, o);
                if (pair_less(ot, best)) best = ot;
            }
            if (lane == 0) red[warp] = best;
            __syncthreads();
            if (tid == 0) {
                for (int w2 = 1; w2 < PAIR_WARPS; ++w2) if (pair_less(red[w2], best)) best = red[w2];
                picked[round] = best.s;
                chosen_s = best.s;
            }
            __syncthreads();
        }
        const int s = chosen_s;
        const int rg = rg_of[s];
        int *v = V + (size_t)rg * LP;
        for (int x = tid; x < LP; x += PAIR_THREADS) v[x] += wb[x];
        if (tid == 0) {
            slot_of[b] = s;
            fillp[s] = 0;
            free_rg[rg] -= 1;
            e_old[rg] += kd[rg];
        }
        __syncthreads();
    }
    for (int i = tid; i < N; i += PAIR_THREADS) lay_out[(size_t)j * N + i] = slot_of[lay[i]];
}

size_t rp_pair_smem_bytes(const RpDims &dm)
{
    return sizeof(i64) * 2 * dm.RG + sizeof(int) * 2 * dm.RG + sizeof(int) * ((size_t)5 * dm.K + 1) + sizeof(int) * (dm.N + 1) +
           sizeof(i64) * dm.K + 16;
}

// Pairs members [first, first + count) of lay_in into lay_out; prof is scratch for `count`
// members ([count][K][LP] ints), V the rank-load cells of the members ([P_pop][RG][LP], overwritten).
int rp_launch_edp_pair(rp_ctx *c, const int *lay_in, int *lay_out, int *prof, int first, int count, int width)
{
    const RpDims &dm = c->dm;
    const size_t smem = rp_pair_smem_bytes(dm);
    if (smem > 200 * 1024) return RP_ERR_RANGE;
    if (smem > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_edp_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const unsigned short *rg_of = (const unsigned short *)(c->d_static + c->sl.off_rg);
    k_edp_pair<<<count, PAIR_THREADS, smem, c->stream>>>(dm, c->d_q, rg_of, lay_in, lay_out, prof, c->d_W, first, width,
                                                         (u32)c->cfg.seed, (u32)(c->cfg.seed >> 32));
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
