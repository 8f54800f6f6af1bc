// Row count R* and the length-only seed layout (Section 3.2 of the paper; first line of
// Algorithm 2), as one CTA on the GPU so that the whole plan stays stream-ordered.
//
// The samples are sorted by (-t_i, i) with a bitonic sort on 64-bit keys, then for
// R = R_lb, R_lb+1, ... first-fit-decreasing is tried into K = R*D cells: the K longest
// samples open the cells, each later sample goes to the lowest-numbered cell it still fits
// in.  The fit search is done by one warp, 32 cells per ballot.
#include "rp_common.cuh"

#define PACK_THREADS 1024

// First fit of the samples keys[K..N) into K cells by one warp; lane `tid` owns cells
// [tid*B, tid*B+B).  Returns true when some sample fits nowhere.  BR >= B cells per lane are
// kept in registers (statically indexed); the shared-memory variant handles any B.
template <int BR>
__device__ __forceinline__ bool first_fit_regs(const RpDims &dm, const u64 *keys, int *fill, int *cell_of, int K, int B, int tid)
{
    const int b0 = tid * B;
    int rem[BR];
    int blockmax = -1;
    bool failed = false;                           // some sample fitted nowhere (the rest of the pass is then moot)
#pragma unroll
    for (int u = 0; u < BR; ++u) {
        rem[u] = (u < B && b0 + u < K) ? dm.C - fill[b0 + u] : -1;
        blockmax = max(blockmax, rem[u]);
    }
    for (int x0 = K; x0 < dm.N; x0 += 32) {
        // the next 32 keys, one per lane, handed out by shuffles
        const u64 mine = (x0 + tid < dm.N) ? keys[x0 + tid] : 0;
        const int nx = min(32, dm.N - x0);
        const int my_len = dm.C - (int)(mine >> 32), my_id = (int)(u32)mine;
#pragma unroll 4
        for (int y = 0; y < nx; ++y) {
            const int ts = __shfl_sync(0xffffffffu, my_len, y), id = __shfl_sync(0xffffffffu, my_id, y);
            // every lane works out what it would do if the sample fell to it (first cell of its
            // block that fits, block maximum afterwards), with no chain from cell to cell; only
            // the ballot and the selects after it link one sample to the next
            bool fits[BR];
#pragma unroll
            for (int u = 0; u < BR; ++u) fits[u] = rem[u] >= ts;
            int first = BR;
#pragma unroll
            for (int u = BR - 1; u >= 0; --u) first = fits[u] ? u : first;
            int nm = -1;
#pragma unroll
            for (int u = 0; u < BR; ++u) nm = max(nm, u == first ? rem[u] - ts : rem[u]);
            const unsigned m = __ballot_sync(0xffffffffu, blockmax >= ts);
            failed |= (m == 0);
            const bool win = (tid == __ffs(m) - 1);
#pragma unroll
            for (int u = 0; u < BR; ++u) rem[u] = (win && u == first) ? rem[u] - ts : rem[u];
            blockmax = win ? nm : blockmax;
            if (win) cell_of[id] = b0 + first;
        }
    }
    return failed;
}

__device__ __forceinline__ bool first_fit_smem(const RpDims &dm, const u64 *keys, int *fill, int *cell_of, int K, int B, int tid)
{
    const int b0 = tid * B, b1 = min(K, b0 + B);
    int blockmax = -1;
    for (int b = b0; b < b1; ++b) blockmax = max(blockmax, dm.C - fill[b]);
    for (int x = K; x < dm.N; ++x) {
        const u64 key = keys[x];
        const int ts = dm.C - (int)(key >> 32);
        const unsigned m = __ballot_sync(0xffffffffu, blockmax >= ts);
        if (!m) return true;
        if (tid == __ffs(m) - 1) {
            int found = -1, nm = -1;
            for (int b = b0; b < b1; ++b) {
                int rem = dm.C - fill[b];
                if (found < 0 && rem >= ts) { found = b; rem -= ts; fill[b] += ts; }
                nm = max(nm, rem);
            }
            blockmax = nm;
            cell_of[(u32)key] = found;
        }
    }
    return false;
}

__global__ void __launch_bounds__(PACK_THREADS)
k_pack_ffd(RpDims dm, const int *__restrict__ t, int min_rows, u64 *__restrict__ keys_g, int n_pow2,
           int *__restrict__ fill_g, int *__restrict__ cell_of, int *__restrict__ out, int *__restrict__ order_out)
{
    extern __shared__ u64 keys_s[];
    u64 *keys = keys_g ? keys_g : keys_s;
    int *fill = fill_g ? fill_g : (int *)(keys_s + (keys_g ? 0 : n_pow2));
    __shared__ i64 total_s;
    __shared__ int fail_s;
    const int tid = threadIdx.x, nt = (int)blockDim.x;
    if (tid == 0) total_s = 0;
    __syncthreads();
    i64 part = 0;
    for (int i = tid; i < n_pow2; i += nt) {
        if (i < dm.N) {
            int ti = t[i];
            part += ti;
            keys[i] = ((u64)(u32)(dm.C - ti) << 32) | (u32)i;     // ascending = longest first, then id
        } else {
            keys[i] = ~0ull;
        }
    }
    for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((tid & 31) == 0 && part) atomicAdd((u64 *)&total_s, (u64)part);
    __syncthreads();
    // Bitonic sort.  Element i sits with thread i % nt, so partners closer than 32 are
    // lanes of one warp: those exchanges run on registers with shuffles (no block-wide barrier),
    // the wider ones through the key array.
    constexpr int SORT_E = 8;                      // elements per thread at most (n_pow2 <= 8192 on this path)
    const bool in_regs = n_pow2 <= SORT_E * nt;
    for (int k = 2; k <= n_pow2; k <<= 1) {
        int j = k >> 1;
        for (; j >= 32 || (j > 0 && !in_regs); j >>= 1) {
            for (int i = tid; i < n_pow2; i += nt) {
                int ixj = i ^ j;
                if (ixj > i) {
                    u64 a = keys[i], b = keys[ixj];
                    bool up = ((i & k) == 0);
                    if ((a > b) == up) { keys[i] = b; keys[ixj] = a; }
                }
            }
            __syncthreads();
        }
        if (j > 0) {
            // all remaining distances of this k (and, while k <= 32, of the following k as well)
            u64 r[SORT_E];
#pragma unroll
            for (int m = 0; m < SORT_E; ++m) { const int i = m * nt + tid; r[m] = i < n_pow2 ? keys[i] : ~0ull; }
            int kk = k;
            for (;;) {
                for (int jj = min(kk >> 1, 16); jj > 0; jj >>= 1) {
#pragma unroll
                    for (int m = 0; m < SORT_E; ++m) {
                        const int i = m * nt + tid;
                        if (m * nt >= n_pow2) break;          // uniform: no element of this slot exists
                        const u64 o = __shfl_xor_sync(0xffffffffu, r[m], jj);
                        const bool up = ((i & kk) == 0), lower = ((tid & jj) == 0);
                        const u64 lo = r[m] < o ? r[m] : o, hi = r[m] < o ? o : r[m];
                        r[m] = (lower == up) ? lo : hi;
                    }
                }
                if (kk >= 32 || (kk << 1) > n_pow2) break;
                kk <<= 1;                                       // the next k still fits inside a warp
            }
            k = kk;
#pragma unroll
            for (int m = 0; m < SORT_E; ++m) { const int i = m * nt + tid; if (i < n_pow2) keys[i] = r[m]; }
            __syncthreads();
        }
    }
    for (int x = tid; x < dm.N; x += nt) order_out[x] = (int)(u32)keys[x];   // samples by (-t, i)
    const i64 cap_row = (i64)dm.C * dm.D;
    i64 Rlb = (total_s + cap_row - 1) / cap_row;
    if (Rlb < 1) Rlb = 1;
    if (Rlb < min_rows) Rlb = min_rows;
    int Rstar = 0;
    for (i64 R = Rlb; R * dm.D <= dm.N && !Rstar; ++R) {
        const int K = (int)(R * dm.D);
        if (tid == 0) fail_s = 0;
        // the K longest samples open the cells
        for (int x = tid; x < K; x += nt) {
            const u64 key = keys[x];
            fill[x] = dm.C - (int)(key >> 32);
            cell_of[(u32)key] = x;
        }
        __syncthreads();
        if (tid < 32) {
            // First fit = the lowest cell whose remaining capacity takes the sample.  Each lane
            // owns a block of B consecutive cells and keeps the largest remaining capacity of its
            // block in a register: one ballot finds the lowest lane that can take the sample, and
            // only that lane scans its block (held in registers when B <= 16).
            const int B = (K + 31) / 32;
            bool failed;
            if (B <= 4) failed = first_fit_regs<4>(dm, keys, fill, cell_of, K, B, tid);
            else if (B <= 8) failed = first_fit_regs<8>(dm, keys, fill, cell_of, K, B, tid);
            else if (B <= 16) failed = first_fit_regs<16>(dm, keys, fill, cell_of, K, B, tid);
            else failed = first_fit_smem(dm, keys, fill, cell_of, K, B, tid);
            if (failed && tid == 0) fail_s = 1;
        }
        __syncthreads();
        if (!fail_s) Rstar = (int)R;
        __syncthreads();
    }
    if (tid == 0) {
        out[0] = Rstar;
        out[1] = (Rstar != 0 && Rstar == Rlb) ? 1 : 0;
        out[2] = (int)(Rlb > 0x7fffffff ? 0x7fffffff : Rlb);
        out[3] = (Rstar == 0);
    }
}

int rp_launch_pack(rp_ctx *c, int /*unused*/) { return rp_launch_pack_on(c, c->stream); }

int rp_launch_pack_on(rp_ctx *c, cudaStream_t stream)
{
    const RpDims &dm = c->dm;
    int n_pow2 = 1;
    while (n_pow2 < dm.N) n_pow2 <<= 1;
    // sort keys (8 bytes each) and cell fills (4 bytes per cell, at most N cells) on chip when they fit
    size_t smem = (size_t)n_pow2 * sizeof(u64) + (size_t)dm.N * sizeof(int);
    u64 *keys_g = nullptr;
    int *fill_g = nullptr;
    if (smem > 160 * 1024) { keys_g = c->d_sort_keys; fill_g = (int *)(c->d_sort_keys + n_pow2); smem = 0; }
    if (smem > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_pack_ffd, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // small windows: fewer warps make the block-wide barriers of the sort cheaper
    const int threads = n_pow2 >= PACK_THREADS ? PACK_THREADS : (n_pow2 < 256 ? 256 : n_pow2);
    k_pack_ffd<<<1, threads, smem, stream>>>(dm, c->d_t, c->cfg.min_rows, keys_g, n_pow2, fill_g,
                                                    c->d_seed_layout, c->d_pack_out, c->d_order);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}
