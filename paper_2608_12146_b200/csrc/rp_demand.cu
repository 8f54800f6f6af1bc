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

// The same pass for rows that are whole multiples of 128 experts (512 bytes) on 16-byte aligned
// tensors.  One CTA owns one layer and a range of samples: its warps take the samples round
// robin, every lane reads 16 bytes of a row, the loads of several rows are issued before any is
// consumed, and a row is summed exactly with two 32-bit warp reductions (low and high 16 bits of
// the counts, neither of which can overflow for E <= 1024; a count outside [0, k*t_i] already
// fails the row).  The warps' column sums meet in shared memory, so the CTA issues one atomic
// per expert.
#define K1V_ROWS_MIN 2
template <int NQ>               // 16-byte pieces per lane and row = E / 128
__global__ void __launch_bounds__(K1_WARPS * 32)
k_check_reduce_vec(const int4 *__restrict__ a, const int *__restrict__ t, RpDims dm, int chunk,
                   i64 *__restrict__ Lagg, int *__restrict__ status, i64 *__restrict__ t_sum)
{
    constexpr int K1V_ROWS = NQ == 1 ? 8 : (NQ == 2 ? 4 : K1V_ROWS_MIN);      // 128 bytes per lane in flight
    extern __shared__ __align__(16) i64 colsum[];          // [K1_WARPS][E]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int l = blockIdx.x % dm.L;
    const int i0 = (blockIdx.x / dm.L) * chunk;
    const int i1 = min(dm.N, i0 + chunk);
    const size_t row4 = (size_t)dm.E >> 2;            // 16-byte pieces per row
    i64 tsum = 0;
    bool bad = false;
    i64 acc[NQ][4];
#pragma unroll
    for (int c = 0; c < NQ; ++c) { acc[c][0] = 0; acc[c][1] = 0; acc[c][2] = 0; acc[c][3] = 0; }
    for (int ib = i0 + warp; ib < i1; ib += K1_WARPS * K1V_ROWS) {
        int4 v[K1V_ROWS][NQ];
        int ti[K1V_ROWS];
#pragma unroll
        for (int r = 0; r < K1V_ROWS; ++r) {
            const int i = min(ib + r * K1_WARPS, i1 - 1);              // past the end: the last row again, not counted
            const int4 *row = a + ((size_t)i * dm.L + l) * row4;
#pragma unroll
            for (int c = 0; c < NQ; ++c) v[r][c] = __ldcs(row + c * 32 + lane);     // read once: streaming
            ti[r] = __ldg(t + i);
        }
#pragma unroll
        for (int r = 0; r < K1V_ROWS; ++r) {
            if (ib + r * K1_WARPS >= i1) break;
            const i64 kt = (i64)dm.k * ti[r];
            const unsigned ktu = kt < 0x7fffffffll ? (kt < 0 ? 0u : (unsigned)kt) : 0x7fffffffu;   // k*C < 2^31 for any window that loads
            tsum += ti[r];
            unsigned part = 0;                         // this lane's share of the row sum, at most k*t once nothing is out of range
            bool out = false;
#pragma unroll
            for (int c = 0; c < NQ; ++c) {
                const unsigned x0 = (unsigned)v[r][c].x, x1 = (unsigned)v[r][c].y, x2 = (unsigned)v[r][c].z, x3 = (unsigned)v[r][c].w;
                // negative counts are huge as unsigned: one comparison covers both ends of [0, k*t]
                out |= (x0 > ktu) | (x1 > ktu) | (x2 > ktu) | (x3 > ktu);
                const unsigned s01 = x0 + x1, s23 = x2 + x3;               // each term below 2^31: no wrap
                out |= (s01 > ktu) | (s23 > ktu);
                const unsigned s4 = s01 + s23;
                out |= (s4 > ktu);
                part += out ? 0u : s4;
                out |= (part > ktu);
                acc[c][0] += v[r][c].x; acc[c][1] += v[r][c].y; acc[c][2] += v[r][c].z; acc[c][3] += v[r][c].w;
            }
            const unsigned slo = __reduce_add_sync(0xffffffffu, out ? 0u : (part & 0xffffu));
            const unsigned shi = __reduce_add_sync(0xffffffffu, out ? 0u : (part >> 16));
            const i64 rs = (i64)slo + ((i64)shi << 16);
            bad |= __any_sync(0xffffffffu, out) || rs != kt || ti[r] < 1 || ti[r] > dm.C;
        }
    }
#pragma unroll
    for (int c = 0; c < NQ; ++c)
#pragma unroll
        for (int u = 0; u < 4; ++u) colsum[(size_t)warp * dm.E + (c * 32 + lane) * 4 + u] = acc[c][u];
    __syncthreads();
    for (int e = threadIdx.x; e < dm.E; e += K1_WARPS * 32) {
        i64 sum = 0;
#pragma unroll
        for (int w = 0; w < K1_WARPS; ++w) sum += colsum[(size_t)w * dm.E + e];
        if (sum) atomicAdd((u64 *)&Lagg[(size_t)l * dm.E + e], (u64)sum);
    }
    if (bad && lane == 0) atomicExch(&status[RP_SW_BAD_SAMPLE], 1);
    if (l == 0 && lane == 0 && tsum > 0) atomicAdd((u64 *)t_sum, (u64)tsum);      // tokens of this warp's samples, once
}

// The same pass as one sequential stream.  A CTA owns a range of samples, i.e. one contiguous
// piece of the tensor; warp w of its NW warps owns the layers w, w + NW, ... (LW of them: L = NW*LW),
// so that the warps of a CTA together read whole samples front to back while every warp keeps the
// column sums of its own layers in registers.  SPI samples are in flight per warp at a time.
template <int NQ, int LW, int NW, int SPI>
__global__ void __launch_bounds__(NW * 32)
k_check_reduce_seq(const int4 *__restrict__ a, const int *__restrict__ t, RpDims dm, int chunk,
                   i64 *__restrict__ Lagg, int *__restrict__ status, i64 *__restrict__ t_sum)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int i0 = blockIdx.x * chunk;
    const int i1 = min(dm.N, i0 + chunk);
    const size_t row4 = (size_t)dm.E >> 2;
    i64 acc[LW][NQ][4];
#pragma unroll
    for (int li = 0; li < LW; ++li)
#pragma unroll
        for (int c = 0; c < NQ; ++c) { acc[li][c][0] = 0; acc[li][c][1] = 0; acc[li][c][2] = 0; acc[li][c][3] = 0; }
    i64 tsum = 0;
    bool bad = false;
    for (int ib = i0; ib < i1; ib += SPI) {
        int4 v[SPI][LW][NQ];
        int ti[SPI];
#pragma unroll
        for (int s = 0; s < SPI; ++s) {
            const int i = min(ib + s, i1 - 1);                       // past the end: the last sample again, not counted
            ti[s] = __ldg(t + i);
#pragma unroll
            for (int li = 0; li < LW; ++li) {
                const int4 *row = a + ((size_t)i * dm.L + warp + li * NW) * row4;
#pragma unroll
                for (int c = 0; c < NQ; ++c) v[s][li][c] = __ldcs(row + c * 32 + lane);
            }
        }
#pragma unroll
        for (int s = 0; s < SPI; ++s) {
            if (ib + s >= i1) break;
            const i64 kt = (i64)dm.k * ti[s];
            const unsigned ktu = kt < 0x7fffffffll ? (kt < 0 ? 0u : (unsigned)kt) : 0x7fffffffu;
            if (warp == 0) tsum += ti[s];
            bad |= ti[s] < 1 || ti[s] > dm.C;
#pragma unroll
            for (int li = 0; li < LW; ++li) {
                unsigned part = 0;
                bool out = false;
#pragma unroll
                for (int c = 0; c < NQ; ++c) {
                    const int4 x = v[s][li][c];
                    const unsigned x0 = (unsigned)x.x, x1 = (unsigned)x.y, x2 = (unsigned)x.z, x3 = (unsigned)x.w;
                    out |= (x0 > ktu) | (x1 > ktu) | (x2 > ktu) | (x3 > ktu);
                    const unsigned s01 = x0 + x1, s23 = x2 + x3;
                    out |= (s01 > ktu) | (s23 > ktu);
                    const unsigned s4 = s01 + s23;
                    out |= (s4 > ktu);
                    part += out ? 0u : s4;
                    out |= (part > ktu);
                    acc[li][c][0] += x.x; acc[li][c][1] += x.y; acc[li][c][2] += x.z; acc[li][c][3] += x.w;
                }
                const unsigned slo = __reduce_add_sync(0xffffffffu, out ? 0u : (part & 0xffffu));
                const unsigned shi = __reduce_add_sync(0xffffffffu, out ? 0u : (part >> 16));
                bad |= __any_sync(0xffffffffu, out) || ((i64)slo + ((i64)shi << 16)) != kt;
            }
        }
    }
#pragma unroll
    for (int li = 0; li < LW; ++li)
#pragma unroll
        for (int c = 0; c < NQ; ++c)
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (acc[li][c][u]) atomicAdd((u64 *)&Lagg[(size_t)(warp + li * NW) * dm.E + (c * 32 + lane) * 4 + u], (u64)acc[li][c][u]);
    if (bad && lane == 0) atomicExch(&status[RP_SW_BAD_SAMPLE], 1);
    if (warp == 0 && lane == 0 && tsum > 0) atomicAdd((u64 *)t_sum, (u64)tsum);
}

template <int NQ, int LW, int NW, int SPI>
static int launch_check_reduce_seq(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    int chunk = (dm.N + 2 * 148 - 1) / (2 * 148);           // two CTAs per SM: enough bytes in flight, few enough atomics
    chunk = chunk < SPI ? SPI : chunk;
    const int grid = (dm.N + chunk - 1) / chunk;
    k_check_reduce_seq<NQ, LW, NW, SPI><<<grid, NW * 32, 0, c->stream>>>((const int4 *)c->d_a, c->d_t, dm, chunk, c->d_Lagg,
                                                                       c->d_status, c->d_counters + 7);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

int rp_launch_check_reduce(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    RP_CUDA(cudaMemsetAsync(c->d_Lagg, 0, sizeof(i64) * dm.L * dm.E, c->stream));
    // The sequential form where it measured faster (512-byte rows, 32 layers: one atomic per expert,
    // layer and CTA is then the smaller part of the time; on wider or fewer rows the form below wins).
    if (((size_t)c->d_a & 15) == 0 && dm.N >= 2 * 148 && dm.E == 128 && dm.L == 32) return launch_check_reduce_seq<1, 2, 16, 4>(c);
    if (dm.E % 128 == 0 && dm.E <= 1024 && ((size_t)c->d_a & 15) == 0) {
        // one CTA per (layer, range of samples): four CTAs per SM (one wave), at least 64 samples each
        int splits = (4 * 148) / dm.L;
        splits = splits < 1 ? 1 : splits;
        int chunk = (dm.N + splits - 1) / splits;
        chunk = chunk < K1_WARPS * 8 ? K1_WARPS * 8 : chunk;
        splits = (dm.N + chunk - 1) / chunk;
        const int grid = splits * dm.L;
        const size_t smem = sizeof(i64) * K1_WARPS * dm.E;
        const int4 *a4 = (const int4 *)c->d_a;
#define K1V_CASE(NQ_)                                                                              \
        do {                                                                                       \
            if (smem > 32 * 1024)                                                                  \
                RP_CUDA(cudaFuncSetAttribute(k_check_reduce_vec<NQ_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
            k_check_reduce_vec<NQ_><<<grid, K1_WARPS * 32, smem, c->stream>>>(a4, c->d_t, dm, chunk, c->d_Lagg, \
                                                                             c->d_status, c->d_counters + 7); \
        } while (0)
        switch (dm.E / 128) {
            case 1: K1V_CASE(1); break;
            case 2: K1V_CASE(2); break;
            case 3: K1V_CASE(3); break;
            case 4: K1V_CASE(4); break;
            case 5: K1V_CASE(5); break;
            case 6: K1V_CASE(6); break;
            case 7: K1V_CASE(7); break;
            default: K1V_CASE(8); break;
        }
#undef K1V_CASE
        ++g_rp_launches;
        RP_CUDA(cudaGetLastError());
        return RP_OK;
    }
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

// The same projection for rows that are whole multiples of 128 experts on 16-byte aligned tensors
// with at most 32 ranks.  One CTA owns one layer and a range of samples, so the layer's inverse
// placement sits in registers (lane (p, part) keeps the PER slots it sums) and no table has to be
// staged.  A warp stages K3V_ROWS rows at a time with 16-byte loads, all issued before any is
// stored; the gather and the coalesced store of the P ranks follow row by row.
#define K3V_ROWS 4
template <int NQ, int PER>
__global__ void __launch_bounds__(K3_WARPS * 32)
k_project_vec(const int4 *__restrict__ a, const int *__restrict__ inv, RpDims dm, int chunk, int *__restrict__ q)
{
    extern __shared__ __align__(16) int smi[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int *rows_s = smi + (size_t)warp * K3V_ROWS * dm.E;
    const int l = blockIdx.x % dm.L;
    const int i0 = (blockIdx.x / dm.L) * chunk;
    const int i1 = min(dm.N, i0 + chunk);
    int parts = 1;
    while (parts * 2 * dm.P <= 32) parts *= 2;
    const int p = lane / parts, part = lane % parts;
    int iv[PER];
#pragma unroll
    for (int x = 0; x < PER; ++x) iv[x] = (p < dm.P) ? __ldg(inv + (size_t)l * dm.E + p * dm.H + part + x * parts) : 0;
    const size_t row4 = (size_t)dm.E >> 2;
    for (int ib = i0 + warp; ib < i1; ib += K3_WARPS * K3V_ROWS) {
        int4 v[K3V_ROWS][NQ];
#pragma unroll
        for (int u = 0; u < K3V_ROWS; ++u) {
            const int i = min(ib + u * K3_WARPS, i1 - 1);
#pragma unroll
            for (int c = 0; c < NQ; ++c) v[u][c] = __ldcs(a + ((size_t)i * dm.L + l) * row4 + c * 32 + lane);
        }
#pragma unroll
        for (int u = 0; u < K3V_ROWS; ++u)
#pragma unroll
            for (int c = 0; c < NQ; ++c) ((int4 *)(rows_s + (size_t)u * dm.E))[c * 32 + lane] = v[u][c];
        __syncwarp();
#pragma unroll
        for (int u = 0; u < K3V_ROWS; ++u) {
            const int i = ib + u * K3_WARPS;
            if (i >= i1) break;
            const int *row_s = rows_s + (size_t)u * dm.E;
            int s = 0;
#pragma unroll
            for (int x = 0; x < PER; ++x) s += row_s[iv[x]];
            for (int o = parts >> 1; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (p < dm.P && part == 0) __stcs(q + ((size_t)i * dm.L + l) * dm.P + p, s);
        }
        __syncwarp();
    }
}

int rp_launch_project(rp_ctx *c)
{
    const RpDims &dm = c->dm;
    {
        int parts = 1;
        while (parts * 2 * dm.P <= 32) parts *= 2;
        const int per = dm.H / parts;
        const bool per_ok = dm.H % parts == 0 && (per == 1 || per == 2 || per == 4 || per == 8 || per == 16);
        const size_t smem_v = (size_t)K3_WARPS * K3V_ROWS * dm.E * sizeof(int);
        if (dm.E % 128 == 0 && dm.E <= 512 && dm.P <= 32 && per_ok && ((size_t)c->d_a & 15) == 0) {
            // one CTA per (layer, range of samples): about eight CTAs per SM, at least 32 samples each
            int splits = (8 * 148 + dm.L - 1) / dm.L;
            int chunk = (dm.N + splits - 1) / splits;
            chunk = chunk < K3_WARPS * K3V_ROWS ? K3_WARPS * K3V_ROWS : chunk;
            splits = (dm.N + chunk - 1) / chunk;
            const int grid = splits * dm.L;
#define K3V_LAUNCH(NQ_, PER_)                                                                                  \
            do {                                                                                               \
                if (smem_v > 32 * 1024)                                                                        \
                    RP_CUDA(cudaFuncSetAttribute(k_project_vec<NQ_, PER_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_v)); \
                k_project_vec<NQ_, PER_><<<grid, K3_WARPS * 32, smem_v, c->stream>>>((const int4 *)c->d_a, c->d_inv, dm, chunk, c->d_q); \
            } while (0)
#define K3V_CASE(NQ_)                                                                                          \
            switch (per) {                                                                                     \
                case 1: K3V_LAUNCH(NQ_, 1); break;                                                             \
                case 2: K3V_LAUNCH(NQ_, 2); break;                                                             \
                case 4: K3V_LAUNCH(NQ_, 4); break;                                                             \
                case 8: K3V_LAUNCH(NQ_, 8); break;                                                             \
                default: K3V_LAUNCH(NQ_, 16); break;                                                           \
            }
            switch (dm.E / 128) {
                case 1: K3V_CASE(1); break;
                case 2: K3V_CASE(2); break;
                case 3: K3V_CASE(3); break;
                default: K3V_CASE(4); break;
            }
#undef K3V_CASE
#undef K3V_LAUNCH
            ++g_rp_launches;
            RP_CUDA(cudaGetLastError());
            return RP_OK;
        }
    }
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
