// Randomized fixed-row seeds (Algorithm 2 of the paper, trial loop): one warp per trial.
//
// WindowShuffle keeps the window of the next `width` samples (decreasing length) in the
// registers of `width` lanes; RandomizedBestFit ranks the cells a sample fits in by one 64-bit
// key (remaining capacity, then sample count, then index: smaller = fuller, fewer, lower) and
// finds the r-th smallest with r+1 warp-wide minimum passes over per-warp cell tables in
// shared memory.  Random words: Philox(h, 0, trial, 4) for the shuffle, (h, 0, trial, 5) for
// the fit, h = position of the sample in the emitted order.
#include "rp_common.cuh"

#define SEED_WARPS 4

// Warp minimum of 64-bit keys with two reduction instructions: the smallest high word, then the
// smallest low word among the lanes that hold it.
__device__ __forceinline__ u64 warp_min_u64(u64 v)
{
    const u32 hi = (u32)(v >> 32), lo = (u32)v;
    const u32 mh = __reduce_min_sync(0xffffffffu, hi);
    const u32 ml = __reduce_min_sync(0xffffffffu, hi == mh ? lo : 0xffffffffu);
    return ((u64)mh << 32) | ml;
}

__global__ void __launch_bounds__(SEED_WARPS * 32)
k_seed_trials(const int *__restrict__ t, const int *__restrict__ order, const int *__restrict__ seed_layout, RpDims dm,
              int width, u32 key0, u32 key1, int Ppop, int *__restrict__ layouts, int *__restrict__ ok)
{
    extern __shared__ int sm[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int *fill = sm + (size_t)warp * 2 * dm.K;        // tokens per cell
    int *cnt = fill + dm.K;                          // samples per cell
    const int j = blockIdx.x * SEED_WARPS + warp;
    if (j >= Ppop) return;
    int *lay = layouts + (size_t)j * dm.N;
    if (j == 0) {                                    // member 0 is the length-only seed
        for (int i = lane; i < dm.N; i += 32) lay[i] = seed_layout[i];
        if (lane == 0) ok[0] = 1;
        return;
    }
    for (int c = lane; c < dm.K; c += 32) { fill[c] = 0; cnt[c] = 0; }
    __syncwarp();
    int win = -1, nwin = 0, next = 0;                // lane x < nwin holds the x-th sample of the window
    bool good = true;
    for (int h = 0; h < dm.N; ++h) {
        while (nwin < width && next < dm.N) {        // refill (one sample per step after the start)
            const int s_new = order[next];
            if (lane == nwin) win = s_new;
            ++nwin; ++next;
        }
        const uint4 xs = rp_philox((u32)h, 0u, (u32)j, 4u, key0, key1);
        const int pos = rp_pick(xs.x, nwin);
        const int s = __shfl_sync(0xffffffffu, win, pos);
        const int up = __shfl_down_sync(0xffffffffu, win, 1);
        if (lane >= pos && lane < nwin - 1) win = up;        // close the gap, order kept
        --nwin;
        const int ts = t[s];
        int b;
        if (h < dm.K) b = h;
        else {
            // feasible cells, ranked by (remaining capacity, count, index)
            int nc = 0;
            for (int c0 = 0; c0 < dm.K; c0 += 32) {
                const int c = c0 + lane;
                nc += __popc(__ballot_sync(0xffffffffu, c < dm.K && fill[c] + ts <= dm.C));
            }
            if (nc == 0) { good = false; break; }
            const uint4 xf = rp_philox((u32)h, 0u, (u32)j, 5u, key0, key1);
            const int r = rp_pick(xf.x, nc < width ? nc : width);
            u64 prev = 0;                            // keys are >= 1: (.., index + 1)
            for (int round = 0; round <= r; ++round) {
                u64 best = ~0ull;
                for (int c = lane; c < dm.K; c += 32) {
                    const int f = fill[c];
                    if (f + ts > dm.C) continue;
                    const u64 key = ((u64)(u32)(dm.C - f) << 40) | ((u64)(u32)cnt[c] << 20) | (u64)(u32)(c + 1);
                    if (key > prev && key < best) best = key;
                }
                prev = warp_min_u64(best);
            }
            b = (int)(prev & 0xFFFFFu) - 1;
        }
        if (lane == 0) { fill[b] += ts; cnt[b] += 1; lay[s] = b; }
        __syncwarp();
    }
    if (!good) for (int i = lane; i < dm.N; i += 32) lay[i] = seed_layout[i];
    if (lane == 0) ok[j] = good ? 1 : 0;
}

int rp_launch_seed_trials(rp_ctx *c, int width, int *layouts, int *ok)
{
    const RpDims &dm = c->dm;
    const size_t smem = sizeof(int) * (size_t)SEED_WARPS * 2 * dm.K;
    if (smem > 200 * 1024) return RP_ERR_RANGE;
    if (smem > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_seed_trials, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = (c->Ppop + SEED_WARPS - 1) / SEED_WARPS;
    k_seed_trials<<<grid, SEED_WARPS * 32, smem, c->stream>>>(c->d_t, c->d_order, c->d_seed_layout, dm, width,
                                                             (u32)c->cfg.seed, (u32)(c->cfg.seed >> 32), c->Ppop, layouts, ok);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// Best member of a scored population (lexicographic, lowest index on ties): becomes the incumbent.
__global__ void __launch_bounds__(1024)
k_pick_best(const i64 *__restrict__ scores, const int *__restrict__ layouts, int n, int N, int *__restrict__ anc,
            int *__restrict__ inc_layout, i64 *__restrict__ inc_score, i64 *__restrict__ best_out)
{
    __shared__ i64 r0[32], r1[32], r2[32];
    __shared__ int rj[32], win;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    i64 b0 = 0x7fffffffffffffffll, b1 = b0, b2 = b0;
    int bj = 0x7fffffff;
    for (int j = tid; j < n; j += 1024) {
        const i64 s0 = scores[3 * (size_t)j], s1 = scores[3 * (size_t)j + 1], s2 = scores[3 * (size_t)j + 2];
        if (rp_lex_less(s0, s1, s2, b0, b1, b2)) { b0 = s0; b1 = s1; b2 = s2; bj = j; }
        anc[j] = j;                                  // every member continues from its own state
    }
    for (int o = 16; o; o >>= 1) {
        const i64 o0 = __shfl_xor_sync(0xffffffffu, b0, o), o1 = __shfl_xor_sync(0xffffffffu, b1, o);
        const i64 o2 = __shfl_xor_sync(0xffffffffu, b2, o);
        const int oj = __shfl_xor_sync(0xffffffffu, bj, o);
        if (rp_lex_less(o0, o1, o2, b0, b1, b2) || (o0 == b0 && o1 == b1 && o2 == b2 && oj < bj)) { b0 = o0; b1 = o1; b2 = o2; bj = oj; }
    }
    if (lane == 0) { r0[warp] = b0; r1[warp] = b1; r2[warp] = b2; rj[warp] = bj; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 32; ++w)
            if (rp_lex_less(r0[w], r1[w], r2[w], b0, b1, b2) || (r0[w] == b0 && r1[w] == b1 && r2[w] == b2 && rj[w] < bj)) {
                b0 = r0[w]; b1 = r1[w]; b2 = r2[w]; bj = rj[w];
            }
        win = bj;
        inc_score[0] = b0; inc_score[1] = b1; inc_score[2] = b2;
        best_out[0] = b0; best_out[1] = b1; best_out[2] = b2;
    }
    __syncthreads();
    const int *src = layouts + (size_t)win * N;
    for (int i = tid; i < N; i += 1024) inc_layout[i] = src[i];
}

int rp_launch_pick_best(rp_ctx *c, const i64 *scores, const int *layouts, int n, i64 *best_score_out)
{
    k_pick_best<<<1, 1024, 0, c->stream>>>(scores, layouts, n, c->dm.N, c->d_anc, c->d_inc_layout, c->d_inc_score, best_score_out);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
