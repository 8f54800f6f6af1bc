// Routing-demand kernels: input checks + aggregate expert load (K1), layer-local LPT
// placement (K2, Algorithm 1 of the paper) and projection of every sample's demand onto
// physical EP ranks (K3, Eq. physical-rank-demand).
//
// K1 and K3 stream the demand tensor a[N][L][E] once each and are bound by HBM bandwidth:
// algorithmic bytes are N*L*E*4 read (+ N*L*P*4 written by K3).  K2 is a few microseconds
// of integer work per layer.
#include "rp_common.cuh"

#define K1_WARPS 8
#define K1_CHUNK_MAX 32        // samples per CTA, at most

// One warp owns one layer of a chunk of samples: it walks the chunk's rows a[i][l][0..E),
// each row read with coalesced 4-byte loads, keeps the column sums of that layer in
// registers (NC = ceil(E/32) columns per lane) and checks every row sum against k*t_i.
template <int NC>
__global__ void __launch_bounds__(K1_WARPS * 32)
k_check_reduce(const int *__restrict__ a, const int *__restrict__ t, RpDims dm, int chunk,
               i64 *__restrict__ Lagg, int *__restrict__ status, i64 *__restrict__ t_sum)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i0 = blockIdx.x * chunk;
    const int i1 = min(dm.N, i0 + chunk);
    i64 tsum = 0;                  // tokens of this chunk (added up by the warp that owns layer 0)
    for (int l = warp; l < dm.L; l += K1_WARPS) {
        i64 acc[NC];
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[c] = 0;
        for (int i = i0; i < i1; ++i) {
            const int *row = a + ((size_t)i * dm.L + l) * dm.E;
            const int ti = t[i];
            if (l == 0) tsum += ti;
            i64 rs = 0;
            bool neg = false;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                int e = c * 32 + lane;
                int v = (e < dm.E) ? __ldg(row + e) : 0;
                neg |= (v < 0);
                acc[c] += v;
                rs += v;
            }
#pragma unroll
            for (int o = 16; o; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
            neg = __any_sync(0xffffffffu, neg);
            bool bad = neg || rs != (i64)dm.k * ti || ti < 1 || ti > dm.C;
            if (bad && lane == 0) atomicExch(&status[RP_SW_BAD_SAMPLE], 1);
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            int e = c * 32 + lane;
            if (e < dm.E && acc[c]) atomicAdd((u64 *)&Lagg[(size_t)l * dm.E + e], (u64)acc[c]);
        }
    }
    if (warp == 0 && lane == 0 && tsum > 0) atomicAdd((u64 *)t_sum, (u64)tsum);
}

int rp_launch_check_reduce(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    RP_CUDA(cudaMemsetAsync(c->d_Lagg, 0, sizeof(i64) * dm.L * dm.E, c->stream));
    // enough CTAs to fill the GPU on small windows, up to 32 samples per CTA on large ones
    int chunk = (dm.N + 2 * 148 - 1) / (2 * 148);
    chunk = chunk < 4 ? 4 : (chunk > K1_CHUNK_MAX ? K1_CHUNK_MAX : chunk);
    int grid = (dm.N + chunk - 1) / chunk;
    int nc = (dm.E + 31) / 32;
#define K1_CASE(NC_)                                                                         \
    k_check_reduce<NC_><<<grid, K1_WARPS * 32, 0, c->stream>>>(c->d_a, c->d_t, dm, chunk, c->d_Lagg, \
                                                               c->d_status, c->d_counters + 7)
    if (nc <= 1) K1_CASE(1);
    else if (nc <= 2) K1_CASE(2);
    else if (nc <= 4) K1_CASE(4);
    else if (nc <= 8) K1_CASE(8);
    else if (nc <= 16) K1_CASE(16);
    else if (nc <= 32) K1_CASE(32);
    else return RP_ERR_RANGE;             // more than 1024 experts per layer
#undef K1_CASE
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// Algorithm 1 for one layer per CTA.  Experts are ranked by (-load, id) by counting how
// many experts precede each one; then one warp assigns them in that order to the rank
// with the smallest (load, id) among ranks holding fewer than H experts.
__global__ void __launch_bounds__(1024)
k_lpt(const i64 *__restrict__ Lagg, RpDims dm, int *__restrict__ pi, int *__restrict__ inv,
      i64 *__restrict__ rank_load)
{
    extern __shared__ unsigned char smraw[];
    i64 *load = (i64 *)smraw;                 // [E]
    i64 *G = load + dm.E;                     // [P]
    int *order = (int *)(G + dm.P);           // [E]
    int *cnt = order + dm.E;                  // [P]
    const int l = blockIdx.x;
    const i64 *Le = Lagg + (size_t)l * dm.E;
    for (int e = threadIdx.x; e < dm.E; e += blockDim.x) load[e] = Le[e];
    for (int p = threadIdx.x; p < dm.P; p += blockDim.x) { G[p] = 0; cnt[p] = 0; }
    __syncthreads();
    for (int e = threadIdx.x; e < dm.E; e += blockDim.x) {
        i64 mine = load[e];
        int before = 0;
        for (int f = 0; f < dm.E; ++f) {
            i64 o = load[f];
            before += (o > mine) || (o == mine && f < e);
        }
        order[before] = e;
    }
    __syncthreads();
    if (threadIdx.x < 32 && dm.P <= 128) {
        // Rank p lives in lane p % 32 (registers: load and slot count).  The least-loaded rank with
        // a free slot is found by three warp reductions: smallest high word of the load, smallest
        // low word among those, lowest rank id among those.
        const int lane = threadIdx.x;
        i64 Gr[4] = { 0, 0, 0, 0 };
        int cr[4] = { 0, 0, 0, 0 };
        for (int x = 0; x < dm.E; ++x) {
            const int e = order[x];
            const i64 le = load[e];
            i64 bG = 0x7fffffffffffffffll;
            int bP = 0x7fffffff;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int p = lane + 32 * u;
                if (p < dm.P && cr[u] < dm.H && Gr[u] < bG) { bG = Gr[u]; bP = p; }      // ascending p: first wins
            }
            const u32 hi = (u32)((u64)bG >> 32);
            const u32 mh = __reduce_min_sync(0xffffffffu, hi);
            const u32 lo = (hi == mh) ? (u32)bG : 0xffffffffu;
            const u32 ml = __reduce_min_sync(0xffffffffu, lo);
            const int cand = (hi == mh && lo == ml) ? bP : 0x7fffffff;
            const int mp = __reduce_min_sync(0xffffffffu, cand);
            if (lane == (mp & 31)) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (u == (mp >> 5)) {
                        const int slot = mp * dm.H + cr[u];
                        pi[(size_t)l * dm.E + e] = slot;
                        inv[(size_t)l * dm.E + slot] = e;
                        Gr[u] += le;
                        cr[u] += 1;
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) { const int p = lane + 32 * u; if (p < dm.P) rank_load[(size_t)l * dm.P + p] = Gr[u]; }
    } else if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int width = 1;                               // lanes that hold ranks, rounded up to a power of two
        while (width < dm.P && width < 32) width <<= 1;
        for (int x = 0; x < dm.E; ++x) {
            const int e = order[x];
            i64 bestG = 0x7fffffffffffffffll;
            int bestP = 0x7fffffff;
            for (int p = lane; p < dm.P; p += 32)
                if (cnt[p] < dm.H && (G[p] < bestG || (G[p] == bestG && p < bestP))) { bestG = G[p]; bestP = p; }
            for (int o = width >> 1; o; o >>= 1) {   // lane 0 ends up with the minimum over lanes 0..width-1
                i64 og = __shfl_xor_sync(0xffffffffu, bestG, o);
                int op = __shfl_xor_sync(0xffffffffu, bestP, o);
                if (og < bestG || (og == bestG && op < bestP)) { bestG = og; bestP = op; }
            }
            if (lane == 0) {
                int slot = bestP * dm.H + cnt[bestP];
                pi[(size_t)l * dm.E + e] = slot;
                inv[(size_t)l * dm.E + slot] = e;
                G[bestP] += load[e];
                cnt[bestP] += 1;
            }
            __syncwarp();
        }
        for (int p = lane; p < dm.P; p += 32) rank_load[(size_t)l * dm.P + p] = G[p];
    }
}

int rp_launch_lpt(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    size_t smem = sizeof(i64) * (dm.E + dm.P) + sizeof(int) * (dm.E + dm.P);
    int threads = dm.E < 32 ? 32 : (dm.E > 1024 ? 1024 : ((dm.E + 31) / 32) * 32);
    k_lpt<<<dm.L, threads, smem, c->stream>>>(c->d_Lagg, dm, c->d_pi, c->d_inv, c->d_rank_load);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

#define K3_WARPS 8
// One warp per (sample, layer) row: the row a[i][l][0..E) is staged in shared memory with
// coalesced loads, then each rank's H experts (slots p*H .. p*H+H-1 through the inverse
// placement) are summed.  Lanes are split (rank, part) so that all 32 lanes gather when
// P < 32; the parts are folded with shuffles.
__global__ void __launch_bounds__(K3_WARPS * 32)
k_project(const int *__restrict__ a, const int *__restrict__ inv, RpDims dm, int *__restrict__ q)
{
    extern __shared__ int smi[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int *row_s = smi + warp * dm.E;
    int *inv_s = smi + K3_WARPS * dm.E;        // [L][E] when it fits (flag below), else global
    const bool inv_in_smem = ((size_t)(K3_WARPS + dm.L) * dm.E * sizeof(int) <= 96 * 1024);
    if (inv_in_smem) {
        for (int x = threadIdx.x; x < dm.L * dm.E; x += blockDim.x) inv_s[x] = inv[x];
        __syncthreads();
    }
    int parts = 1;
    while (parts * 2 * dm.P <= 32) parts *= 2;   // largest power of two with P*parts <= 32
    const long long rows = (long long)dm.N * dm.L;
    for (long long r = (long long)blockIdx.x * K3_WARPS + warp; r < rows; r += (long long)gridDim.x * K3_WARPS) {
        const int l = (int)(r % dm.L);
        const int *src = a + (size_t)r * dm.E;
        for (int e = lane; e < dm.E; e += 32) row_s[e] = __ldg(src + e);
        __syncwarp();
        const int *iv = inv_in_smem ? (inv_s + l * dm.E) : (inv + (size_t)l * dm.E);
        for (int p0 = 0; p0 < dm.P; p0 += 32 / parts) {
            int p = p0 + lane / parts, part = lane % parts;
            int s = 0;
            if (p < dm.P)
                for (int n = part; n < dm.H; n += parts) s += row_s[iv[p * dm.H + n]];
            for (int o = parts >> 1; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (p < dm.P && part == 0) q[(size_t)r * dm.P + p] = s;
        }
        __syncwarp();
    }
}

int rp_launch_project(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    size_t smem = (size_t)K3_WARPS * dm.E * sizeof(int);
    if ((size_t)(K3_WARPS + dm.L) * dm.E * sizeof(int) <= 96 * 1024) smem += (size_t)dm.L * dm.E * sizeof(int);
    if (smem > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_project, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long rows = (long long)dm.N * dm.L;
    long long want = (rows + K3_WARPS - 1) / K3_WARPS;
    int grid = (int)(want < 148 * 8 ? want : 148 * 8);
    if (grid < 1) grid = 1;
    k_project<<<grid, K3_WARPS * 32, smem, c->stream>>>(c->d_a, c->d_inv, dm, c->d_q);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
