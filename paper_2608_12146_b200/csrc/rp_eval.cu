// Full evaluation of layouts (K4): cell statistics, per-row-shard rank loads W, expert and
// attention costs, shard work and the score tuple (Sections 3.4-3.5 of the paper).
//
// One CTA per layout.  Samples are bucketed by row-shard in shared memory; each warp then
// owns whole row-shards and adds up the q rows of its members with coalesced loads (q is
// shared by all layouts and stays L2-resident), so W is produced without atomics and is
// written at most once.  Algorithmic bytes per layout: N*2 (assignment) + N*L*P*4 (q rows,
// L2-served) read, R*G*L*P*4 written when W is kept.
#include "rp_score.cuh"

#define EVAL_THREADS 256

__global__ void k_layouts_to_cells(const int *__restrict__ layouts, long long total, int K,
                                   unsigned short *__restrict__ cells, int *__restrict__ status)
{
    long long x = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= total) return;
    int c = layouts[x];
    if (c < 0 || c >= K) { atomicExch(&status[RP_SW_BAD_LAYOUT], 1); c = 0; }
    cells[x] = (unsigned short)c;
}

int rp_launch_cells_from_layouts(rp_ctx *c, const int *layouts, int n, unsigned short *cells)
{
    long long total = (long long)n * c->dm.N;
    int grid = (int)((total + 255) / 256);
    k_layouts_to_cells<<<grid, 256, 0, c->stream>>>(layouts, total, c->dm.K, cells, c->d_status);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// grid = (layouts, splits): the CTAs of a layout share its row-shards (8 per CTA, one per warp);
// the CTA that finishes last (atomic ticket) gathers the row-shard sums and scores the layout.
// DEEP: eight members' loads in flight per pass (few layouts: latency matters); otherwise two
// (many layouts: the CTAs in flight hide the latency and registers are better spent on occupancy).
template <bool DEEP>
__global__ void __launch_bounds__(EVAL_THREADS)
k_eval(const unsigned short *__restrict__ cells, const int *__restrict__ t, const int *__restrict__ q,
       const int *__restrict__ edp, const int *__restrict__ dp_list, const int *__restrict__ dp_off,
       RpDims dm, RpBlob bl, int *__restrict__ W_out, char *__restrict__ blob_out,
       i64 *__restrict__ score_out, double *__restrict__ f64_out, i64 *__restrict__ Esum_g,
       int *__restrict__ tickets)
{
    extern __shared__ __align__(16) unsigned char smraw[];
    // layout: Q[K] u64 | Esum[RG] | Afx[RG] | U[G] | T[K] | cnt[K] | off[RG+1] | cur[RG] | members[N] | cell_of[N]
    u64 *Q = (u64 *)smraw;
    i64 *Esum = (i64 *)(Q + dm.K);
    i64 *Afx = Esum + dm.RG;
    i64 *U = Afx + dm.RG;
    int *T = (int *)(U + dm.G);
    int *cnt = T + dm.K;
    int *off = cnt + dm.K;
    int *cur = off + dm.RG + 1;
    int *members = cur + dm.RG;
    unsigned short *cell_of = (unsigned short *)(members + dm.N);
    __shared__ int last_s;
    RpSmemState st = { cell_of, T, Q, cnt, Esum, Afx, U };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = EVAL_THREADS / 32;
    const int lay = blockIdx.x;
    const unsigned short *src = cells + (size_t)lay * dm.N;
    for (int i = tid; i < dm.N; i += EVAL_THREADS) cell_of[i] = src[i];
    for (int c = tid; c < dm.K; c += EVAL_THREADS) { T[c] = 0; Q[c] = 0; cnt[c] = 0; }
    for (int x = tid; x <= dm.RG; x += EVAL_THREADS) { off[x] = 0; if (x < dm.RG) cur[x] = 0; }
    __syncthreads();
    rp_accumulate_cells(dm, st, t, tid, EVAL_THREADS);
    for (int i = tid; i < dm.N; i += EVAL_THREADS) atomicAdd(&off[rp_rowshard(dm, edp, cell_of[i]) + 1], 1);
    __syncthreads();
    if (tid == 0) for (int x = 0; x < dm.RG; ++x) off[x + 1] += off[x];
    __syncthreads();
    for (int i = tid; i < dm.N; i += EVAL_THREADS) {
        int rg = rp_rowshard(dm, edp, cell_of[i]);
        members[off[rg] + atomicAdd(&cur[rg], 1)] = i;
    }
    __syncthreads();
    i64 *esum_lay = Esum_g + (size_t)lay * dm.RG;
    for (int rg = blockIdx.y * nwarps + warp; rg < dm.RG; rg += gridDim.y * nwarps) {
        const int m0 = off[rg], m1 = off[rg + 1];
        int *wout = W_out ? W_out + ((size_t)lay * dm.RG + rg) * dm.LP : nullptr;
        i64 es;
        if (dm.P <= 32 && (dm.P & (dm.P - 1)) == 0) {
            // four strips of 32 columns at a time: four independent loads per member in flight, the
            // busiest rank of a layer by segmented shuffles over the coalesced column order
            es = 0;
            for (int x0 = 0; x0 < dm.LP; x0 += 128) {
                int acc[4] = { 0, 0, 0, 0 };
                if constexpr (DEEP) {
                    for (int mb = m0; mb < m1; mb += 8) {      // eight members' loads in flight before any is added
                        int v[8][4];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const bool on = mb + e < m1;
                            const int *row = q + (size_t)(on ? members[mb + e] : 0) * dm.LP + x0 + lane;
#pragma unroll
                            for (int u = 0; u < 4; ++u) v[e][u] = (on && x0 + 32 * u + lane < dm.LP) ? __ldg(row + 32 * u) : 0;
                        }
#pragma unroll
                        for (int e = 0; e < 8; ++e)
#pragma unroll
                            for (int u = 0; u < 4; ++u) acc[u] += v[e][u];
                    }
                } else {
#pragma unroll 2
                    for (int m = m0; m < m1; ++m) {
                        const int *row = q + (size_t)members[m] * dm.LP + x0 + lane;
#pragma unroll
                        for (int u = 0; u < 4; ++u) if (x0 + 32 * u + lane < dm.LP) acc[u] += __ldg(row + 32 * u);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int x = x0 + 32 * u + lane;
                    int v = (x < dm.LP) ? acc[u] : 0;
                    if (wout && x < dm.LP) wout[x] = v;
                    for (int o = dm.P >> 1; o; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
                    if ((lane & (dm.P - 1)) == 0 && x < dm.LP) es += v;
                }
            }
            for (int o = 16; o; o >>= 1) es += __shfl_xor_sync(0xffffffffu, es, o);
        } else {
            es = rp_warp_layer_max_sum(dm, lane, [&](int x) {
                int s = 0;
                for (int m = m0; m < m1; ++m) s += __ldg(q + (size_t)members[m] * dm.LP + x);
                if (wout) wout[x] = s;
                return s;
            });
        }
        if (lane == 0) esum_lay[rg] = es;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int ticket = atomicAdd(&tickets[lay], 1);
        last_s = (ticket == (int)gridDim.y - 1);
        if (last_s) tickets[lay] = 0;                 // ready for the next launch
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    for (int rg = tid; rg < dm.RG; rg += EVAL_THREADS) Esum[rg] = ((volatile i64 *)esum_lay)[rg];
    __syncthreads();
    i64 sc[3];
    rp_rows_to_score(dm, st, dp_list, dp_off, tid, EVAL_THREADS, sc);
    if (blob_out) {      // the chain-state blob of this layout (see RpBlob)
        char *b = blob_out + (size_t)lay * bl.bytes;
        for (int c = tid; c < dm.K; c += EVAL_THREADS) {
            ((u64 *)(b + bl.off_Q))[c] = Q[c];
            ((int *)(b + bl.off_T))[c] = T[c];
            ((int *)(b + bl.off_cnt))[c] = cnt[c];
        }
        for (int rg = tid; rg < dm.RG; rg += EVAL_THREADS) {
            ((i64 *)(b + bl.off_Esum))[rg] = Esum[rg];
            ((i64 *)(b + bl.off_Afx))[rg] = Afx[rg];
            ((i64 *)(b + bl.off_Jfx))[rg] = Afx[rg] + dm.EC * Esum[rg];
        }
        for (int g = tid; g < dm.G; g += EVAL_THREADS) ((i64 *)(b + bl.off_U))[g] = U[g];
        if (bl.off_wtab >= 0)          // W_out holds layout `lay` as RG consecutive slices of the pool
            for (int rg = tid; rg < dm.RG; rg += EVAL_THREADS) ((int *)(b + bl.off_wtab))[rg] = lay * dm.RG + rg;
        for (int i = tid; i < dm.N; i += EVAL_THREADS) ((unsigned short *)(b + bl.off_cell))[i] = cell_of[i];
        if (tid == 0) {
            i64 *S = (i64 *)(b + bl.off_S);
            S[0] = sc[0]; S[1] = sc[1]; S[2] = sc[2]; S[3] = rp_energy(sc[0], sc[1], sc[2]);
        }
    }
    if (tid == 0) {
        for (int x = 0; x < 3; ++x) {
            if (score_out) score_out[(size_t)lay * 3 + x] = sc[x];
            if (f64_out) f64_out[(size_t)lay * 3 + x] = (double)sc[x] / (double)dm.SC;
        }
    }
}

static size_t eval_smem_bytes(const RpDims &dm)
{
    size_t b = sizeof(u64) * dm.K + sizeof(i64) * (2 * (size_t)dm.RG + dm.G);
    b += sizeof(int) * (2 * (size_t)dm.K + 2 * (size_t)dm.RG + 1 + dm.N);
    b += sizeof(unsigned short) * dm.N;
    return (b + 15) & ~(size_t)15;
}

int rp_launch_eval(rp_ctx *c, const unsigned short *cells, int n, int *W_out, char *blob_out,
                   i64 *score_out, double *f64_out)
{
    const RpDims &dm = c->dm;
    size_t smem = eval_smem_bytes(dm);
    if (smem > 220 * 1024) return RP_ERR_RANGE;
    if (smem > 32 * 1024) {
        RP_CUDA(cudaFuncSetAttribute(k_eval<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RP_CUDA(cudaFuncSetAttribute(k_eval<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    }
    // few layouts: split each one's row-shards over several CTAs so the GPU is not left idle
    int splits = (2 * 148 + n - 1) / n;
    const int max_splits = (dm.RG + EVAL_THREADS / 32 - 1) / (EVAL_THREADS / 32);
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    if ((long long)n * splits <= 2 * 148)
        k_eval<true><<<dim3(n, splits), EVAL_THREADS, smem, c->stream>>>(cells, c->d_t, c->d_q, c->d_edp, c->d_dp_list, c->d_dp_off,
                                                                        dm, c->bl, W_out, blob_out, score_out, f64_out,
                                                                        c->d_eval_Esum, c->d_eval_tickets);
    else
        k_eval<false><<<dim3(n, splits), EVAL_THREADS, smem, c->stream>>>(cells, c->d_t, c->d_q, c->d_edp, c->d_dp_list, c->d_dp_off,
                                                                         dm, c->bl, W_out, blob_out, score_out, f64_out,
                                                                         c->d_eval_Esum, c->d_eval_tickets);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// ---------------------------------------------------------------------------------------------
// Layout of the chain-state blob and of the per-plan static tables; the static block itself.
// ---------------------------------------------------------------------------------------------
void rp_make_layouts(const RpDims &dm, RpBlob *bl, RpStatic *sl)
{
    int o = 0;
    bl->off_Q = o;    o += 8 * dm.K;
    bl->off_Esum = o; o += 8 * dm.RG;
    bl->off_Afx = o;  o += 8 * dm.RG;
    bl->off_Jfx = o;  o += 8 * dm.RG;
    bl->off_U = o;    o += 8 * dm.G;
    bl->off_S = o;    o += 8 * 4;
    bl->off_T = o;    o += 4 * dm.K;
    bl->off_cnt = o;  o += 4 * dm.K;
    bl->off_cell = o; o += 2 * dm.N;
    bl->off_wtab = -1;
    if (rp_uses_slices(dm)) { o = (o + 3) & ~3; bl->off_wtab = o; o += 4 * dm.RG; }
    bl->bytes = (o + 15) & ~15;
    sl->t_staged = dm.N <= 2048;
    o = 0;
    sl->off_dpl = o;  o += 4 * dm.D;
    sl->off_dpo = o;  o += 4 * (dm.G + 1);
    sl->off_t = o;    o += sl->t_staged ? 4 * dm.N : 0;
    sl->off_rg = o;   o += 2 * dm.K;
    sl->off_g = o;    o += 2 * dm.K;
    sl->off_row = o;  o += 2 * dm.K;
    sl->bytes = (o + 15) & ~15;
}

__global__ void k_build_static(const int *__restrict__ t, const int *__restrict__ edp, const int *__restrict__ dp_list,
                               const int *__restrict__ dp_off, RpDims dm, RpStatic sl, char *__restrict__ blk)
{
    const int tid = blockIdx.x * blockDim.x + threadIdx.x, nt = gridDim.x * blockDim.x;
    for (int d = tid; d < dm.D; d += nt) ((int *)(blk + sl.off_dpl))[d] = dp_list[d];
    for (int g = tid; g <= dm.G; g += nt) ((int *)(blk + sl.off_dpo))[g] = dp_off[g];
    if (sl.t_staged) for (int i = tid; i < dm.N; i += nt) ((int *)(blk + sl.off_t))[i] = t[i];
    for (int c = tid; c < dm.K; c += nt) {
        const int r = c / dm.D, g = edp[c % dm.D];
        ((unsigned short *)(blk + sl.off_rg))[c] = (unsigned short)(r * dm.G + g);
        ((unsigned short *)(blk + sl.off_g))[c] = (unsigned short)g;
        ((unsigned short *)(blk + sl.off_row))[c] = (unsigned short)(r * dm.D);
    }
}

int rp_launch_build_static(rp_ctx *c)
{
    k_build_static<<<4, 256, 0, c->stream>>>(c->d_t, c->d_edp, c->d_dp_list, c->d_dp_off, c->dm, c->sl, c->d_static);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    return RP_OK;
}

// ---------------------------------------------------------------------------------------------
// Load-balance diagnostics (evaluation section of the paper): coefficient of variation of the
// aggregate rank loads, EP peak sum, tail peak, EP balance efficiency, attention and joint proxies.
// ---------------------------------------------------------------------------------------------
struct RpDiagDev { double cv_identity, cv_placed; i64 s_ep, t_ep, n_ep; i64 afx_sum, s0; };

// One thread per layer, each with plain sequential IEEE sums (no fused multiply-add), then
// thread 0 averages the layers in order.
__global__ void k_diag_cv(const i64 *__restrict__ Lagg, const i64 *__restrict__ rank_load, RpDims dm,
                          RpDiagDev *__restrict__ out)
{
    extern __shared__ double cvs[];          // [2][L]
    const int l = threadIdx.x;
    if (l < dm.L) {
        for (int which = 0; which < 2; ++which) {
            double mean = 0.0;
            for (int p = 0; p < dm.P; ++p) {
                i64 g = 0;
                if (which) g = rank_load[(size_t)l * dm.P + p];
                else for (int n = 0; n < dm.H; ++n) g += Lagg[(size_t)l * dm.E + p * dm.H + n];
                mean = __dadd_rn(mean, (double)g);
            }
            mean = __ddiv_rn(mean, (double)dm.P);
            double var = 0.0;
            for (int p = 0; p < dm.P; ++p) {
                i64 g = 0;
                if (which) g = rank_load[(size_t)l * dm.P + p];
                else for (int n = 0; n < dm.H; ++n) g += Lagg[(size_t)l * dm.E + p * dm.H + n];
                const double d = __dsub_rn((double)g, mean);
                var = __dadd_rn(var, __dmul_rn(d, d));
            }
            var = __ddiv_rn(var, (double)dm.P);
            cvs[which * dm.L + l] = (mean > 0.0) ? __ddiv_rn(__dsqrt_rn(var), mean) : 0.0;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0;
        for (int x = 0; x < dm.L; ++x) { a = __dadd_rn(a, cvs[x]); b = __dadd_rn(b, cvs[dm.L + x]); }
        out->cv_identity = __ddiv_rn(a, (double)dm.L);
        out->cv_placed = __ddiv_rn(b, (double)dm.L);
    }
}

// One warp per (row, layer): lanes over ranks, loop over shards; integer results by atomics.
__global__ void k_diag_peaks(const int *__restrict__ W, const char *__restrict__ blob, RpBlob bl, RpDims dm,
                             RpDiagDev *__restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = (gridDim.x * blockDim.x) >> 5;
    i64 s_ep = 0, n_ep = 0, t_ep = 0;
    for (int rl = wid; rl < dm.R * dm.L; rl += nw) {
        const int r = rl / dm.L, l = rl % dm.L;
        i64 peak = 0, best_sum = 0;
        for (int g = 0; g < dm.G; ++g) {
            const int *w = W + (((size_t)r * dm.G + g) * dm.L + l) * dm.P;
            i64 sum = 0, mx = 0;
            for (int p = lane; p < dm.P; p += 32) { const i64 v = w[p]; sum += v; mx = v > mx ? v : mx; }
            for (int o = 16; o; o >>= 1) {
                sum += __shfl_xor_sync(0xffffffffu, sum, o);
                const i64 x = __shfl_xor_sync(0xffffffffu, mx, o);
                mx = x > mx ? x : mx;
            }
            peak = mx > peak ? mx : peak;
            best_sum = sum > best_sum ? sum : best_sum;
        }
        s_ep += peak; n_ep += best_sum; t_ep = peak > t_ep ? peak : t_ep;
    }
    if (lane == 0) {
        if (s_ep) atomicAdd((u64 *)&out->s_ep, (u64)s_ep);
        if (n_ep) atomicAdd((u64 *)&out->n_ep, (u64)n_ep);
        atomicMax((i64 *)&out->t_ep, t_ep);
    }
    if (blockIdx.x == 0 && threadIdx.x < 32) {      // attention total and joint from the layout's blob
        const i64 *Afx = (const i64 *)(blob + bl.off_Afx);
        i64 a = 0;
        for (int x = lane; x < dm.RG; x += 32) a += Afx[x];
        for (int o = 16; o; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) { out->afx_sum = a; out->s0 = ((const i64 *)(blob + bl.off_S))[0]; }
    }
}

extern "C" int rp_diagnostics(rp_ctx *c, const int32_t *layout, rp_diag *out)
{
    if (!c || !out) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    const RpDims &dm = c->dm;
    if (dm.L > 1024) return RP_ERR_RANGE;
    cudaMemPool_t pool;
    RP_TRY(rp_get_pool(c->device, &pool));
    // scratch: cells, W, one blob, the result record, and the row-shard sums / ticket of the scoring kernel
    const size_t wn = (size_t)dm.RG * dm.LP;
    size_t off_cells = 0, off_lay = off_cells + (((size_t)dm.N * 2 + 255) & ~(size_t)255);
    size_t off_W = off_lay + (((size_t)dm.N * 4 + 255) & ~(size_t)255);
    size_t off_blob = off_W + ((wn * 4 + 255) & ~(size_t)255);
    size_t off_res = off_blob + (((size_t)c->bl.bytes + 255) & ~(size_t)255);
    size_t off_es = off_res + 256, off_tk = off_es + (((size_t)dm.RG * 8 + 255) & ~(size_t)255);
    size_t total = off_tk + 256;
    char *buf = nullptr;
    RP_CUDA(cudaMallocFromPoolAsync((void **)&buf, total, pool, c->stream));
    int st = RP_OK;
    cudaError_t e = cudaSuccess;
    do {
        const int *dl = c->d_inc_layout;
        if (layout) {
            e = cudaMemcpyAsync(buf + off_lay, layout, sizeof(int) * dm.N, cudaMemcpyDefault, c->stream);
            if (e != cudaSuccess) break;
            dl = (const int *)(buf + off_lay);
        }
        e = cudaMemsetAsync(buf + off_res, 0, 256 + (off_tk - off_es) + 256, c->stream);
        if (e != cudaSuccess) break;
        e = cudaMemsetAsync(c->d_status + RP_SW_BAD_LAYOUT, 0, sizeof(int), c->stream);
        if (e != cudaSuccess) break;
        k_layouts_to_cells<<<(dm.N + 255) / 256, 256, 0, c->stream>>>(dl, dm.N, dm.K, (unsigned short *)(buf + off_cells),
                                                                     c->d_status);
        ++g_rp_launches;
        const size_t smem = eval_smem_bytes(dm);
        if (smem > 220 * 1024) { st = RP_ERR_RANGE; break; }
        if (smem > 32 * 1024) {
            e = cudaFuncSetAttribute(k_eval<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) break;
        }
        int splits = 2 * 148;
        const int max_splits = (dm.RG + EVAL_THREADS / 32 - 1) / (EVAL_THREADS / 32);
        if (splits > max_splits) splits = max_splits;
        k_eval<true><<<dim3(1, splits), EVAL_THREADS, smem, c->stream>>>((const unsigned short *)(buf + off_cells), c->d_t, c->d_q,
                                                                  c->d_edp, c->d_dp_list, c->d_dp_off, dm, c->bl,
                                                                  (int *)(buf + off_W), buf + off_blob, nullptr, nullptr,
                                                                  (i64 *)(buf + off_es), (int *)(buf + off_tk));
        ++g_rp_launches;
        RpDiagDev *res = (RpDiagDev *)(buf + off_res);
        k_diag_cv<<<1, ((dm.L + 31) / 32) * 32, sizeof(double) * 2 * dm.L, c->stream>>>(c->d_Lagg, c->d_rank_load, dm, res);
        ++g_rp_launches;
        k_diag_peaks<<<148, 256, 0, c->stream>>>((const int *)(buf + off_W), buf + off_blob, c->bl, dm, res);
        ++g_rp_launches;
        e = cudaGetLastError();
        if (e != cudaSuccess) break;
        RpDiagDev h;
        int bad = 0;
        e = cudaMemcpyAsync(&h, res, sizeof h, cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, c->d_status + RP_SW_BAD_LAYOUT, sizeof(int), cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        if (e != cudaSuccess) break;
        if (bad) { st = RP_ERR_ARG; break; }
        out->cv_identity = h.cv_identity; out->cv_placed = h.cv_placed;
        out->s_ep = h.s_ep; out->t_ep = h.t_ep; out->n_ep = h.n_ep;
        out->eta_ep = h.s_ep > 0 ? (double)h.n_ep / ((double)dm.P * (double)h.s_ep) : 1.0;
        out->attention = (double)h.afx_sum / (double)dm.SC;
        out->joint = (double)h.s0 / (double)dm.SC;
    } while (0);
    cudaFreeAsync(buf, c->stream);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return st;
}

// ---------------------------------------------------------------------------------------------
// Scoring layouts without allocating: the kernels above, with their scratch (16-bit cell ids,
// row-shard sums, arrival counters) taken from a fixed array that is part of the library image
// instead of from the context's allocator.
// ---------------------------------------------------------------------------------------------
#define RP_NOALLOC_MAX_LAYOUTS 1024            // layouts per call
#define RP_NOALLOC_MAX_CELLS (1 << 19)         // n * N          (1 MiB of 16-bit cell ids)
#define RP_NOALLOC_MAX_ROWSHARDS (1 << 15)     // n * R * G      (256 KiB of 64-bit sums)

struct RpNoAllocScratch {
    i64 esum[RP_NOALLOC_MAX_ROWSHARDS];
    int tickets[RP_NOALLOC_MAX_LAYOUTS];
    unsigned short cells[RP_NOALLOC_MAX_CELLS];
};
// About 1.3 MiB on every GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(RpNoAllocScratch)];
// Device address of the array above, per device (in host code the symbol itself is only a
// stand-in, never a device address).
static void *g_noalloc_addr[64];

extern "C" int rp_eval_layouts_noalloc(rp_ctx *c, const int32_t *layouts, int32_t n, int64_t *score_fx,
                                       double *score_f64)
{
    if (!c || !layouts || n < 1) return RP_ERR_ARG;
    if (c->stage < 3) return RP_ERR_STATE;
    const RpDims &dm = c->dm;
    if (n > RP_NOALLOC_MAX_LAYOUTS || (long long)n * dm.N > RP_NOALLOC_MAX_CELLS ||
        (long long)n * dm.RG > RP_NOALLOC_MAX_ROWSHARDS)
        return RP_ERR_RANGE;                  // beyond the fixed scratch: use rp_eval_population
    const size_t smem = eval_smem_bytes(dm);
    if (smem > 220 * 1024) return RP_ERR_RANGE;   // nothing has been queued yet
    int cur = -1;
    RP_CUDA(cudaGetDevice(&cur));
    if (cur != c->device || cur < 0 || cur >= 64) return RP_ERR_STATE;
    // every array must already be on the device: staging a host array would need memory
    const void *ptrs[3] = { layouts, score_fx, score_f64 };
    for (int x = 0; x < 3; ++x) {
        if (!ptrs[x]) continue;
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, ptrs[x]) != cudaSuccess) { cudaGetLastError(); return RP_ERR_ARG; }
        if (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) return RP_ERR_ARG;
        if (at.type == cudaMemoryTypeDevice && at.device != c->device) return RP_ERR_ARG;    // another GPU's memory
    }
    if (!g_noalloc_addr[cur]) {               // set-up, once per device, with that device current
        void *p = nullptr;
        RP_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_noalloc_addr[cur] = p;
    }
    RpNoAllocScratch *sc = (RpNoAllocScratch *)g_noalloc_addr[cur];
    // the array keeps what the previous call left: the arrival counters must start at zero
    RP_CUDA(cudaMemsetAsync(sc->tickets, 0, sizeof(int) * n, c->stream));
    RP_CUDA(cudaMemsetAsync(c->d_status + RP_SW_BAD_LAYOUT, 0, sizeof(int), c->stream));
    const long long total = (long long)n * dm.N;
    k_layouts_to_cells<<<(int)((total + 255) / 256), 256, 0, c->stream>>>(layouts, total, dm.K, sc->cells, c->d_status);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    if (smem > 32 * 1024)
        RP_CUDA(cudaFuncSetAttribute(k_eval<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int splits = (2 * 148 + n - 1) / n;
    const int max_splits = (dm.RG + EVAL_THREADS / 32 - 1) / (EVAL_THREADS / 32);
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    k_eval<false><<<dim3(n, splits), EVAL_THREADS, smem, c->stream>>>(sc->cells, c->d_t, c->d_q, c->d_edp, c->d_dp_list, c->d_dp_off,
                                                              dm, c->bl, nullptr, nullptr, (i64 *)score_fx, score_f64, sc->esum,
                                                              sc->tickets);
    ++g_rp_launches;
    RP_CUDA(cudaGetLastError());
    int bad = 0;
    RP_CUDA(cudaMemcpyAsync(&bad, c->d_status + RP_SW_BAD_LAYOUT, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    RP_CUDA(cudaStreamSynchronize(c->stream));
    return bad ? RP_ERR_ARG : RP_OK;
}
