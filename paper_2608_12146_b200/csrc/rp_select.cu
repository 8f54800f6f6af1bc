// Canonicalize, CanonicalMap and QualityDiversitySelect (Section 4.1.1, Algorithm 2) over the
// population as the candidate set.
//
//   signature   a cell is named by its smallest sample; inside a row the cells of one EDP shard
//               are listed by name over the shard's slots (increasing slot), rows are listed by
//               their smallest sample.  Equal signatures = same plan up to row order and
//               exchangeable slots.  A 64-bit hash of the signature finds the candidates for an
//               exact comparison.
//   map         the representative of a class has the lowest score, then the lowest index.
//   distance    Q20 units: cell co-assignment + row co-assignment (1 - pairs together in both /
//               pairs together in either) + sketch distance
//               floor(16 * sum_k sum_r |phi_k(x)[r] - phi_k(y)[r]| / (n_proj * R * F)),
//               phi_k = sorted projection of the Q16 row features (tokens / (C*D), squared
//               lengths / (C*C*D), busiest rank of every (shard, layer) / (k*C*|D_g|)) onto the
//               +-1 vector whose f-th sign is the top bit of Philox(f, 0, k, 7).x.
//   selection   starts from the lowest score; then the representative maximising
//               (distance to the nearest selected one) - ((eta_q16 * gap) >> 16), gap =
//               floor((S0 - S0*) * 2^20 / S0*), ties by lower index.
#include "rp_common.cuh"

#define SEL_THREADS 256
#define SEL_TABLE 4096

struct SelBuf {                 // per-member arrays in global memory
    int *lay;                   // [P][N] layouts
    int *canon;                 // [P][N] signatures
    u64 *hash;                  // [P]
    int *clist, *cstart;        // [P][N], [P][K+1] samples grouped by cell
    int *rlist, *rstart;        // [P][N], [P][R+1] samples grouped by row
    i64 *pc, *pr;               // [P] pairs together in a cell / in a row
    i64 *phi;                   // [P][n_proj][R] sorted projections
};

__device__ __forceinline__ u64 sel_mix(u64 x)
{
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

// ---- signs of the projections: sgn[k][f] = 1 where the entry is -1 -----------------------------
__global__ void k_sel_signs(int F, int n_proj, u32 key0, u32 key1, unsigned char *__restrict__ sgn)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= F * n_proj) return;
    const int k = x / F, f = x % F;
    sgn[x] = (unsigned char)(rp_philox((u32)f, 0u, (u32)k, 7u, key0, key1).x >> 31);
}

// ---- per member: signature, hash, groupings, sketch ---------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS)
k_sel_prepare(RpDims dm, RpBlob bl, const char *__restrict__ blobs, const int *__restrict__ anc,
              const int *__restrict__ W_all, const int *__restrict__ wloc, const unsigned short *__restrict__ g_of_cell,
              const unsigned char *__restrict__ sgn, int n_proj, SelBuf B)
{
    extern __shared__ __align__(16) unsigned char sel_smem[];
    const int N = dm.N, K = dm.K, R = dm.R, D = dm.D, G = dm.G, L = dm.L, P = dm.P;
    const int F = 2 + G * L;
    i64 *ph = (i64 *)sel_smem;                     // [n_proj][R] projections
    int *name = (int *)(ph + (size_t)n_proj * R);  // [K] smallest sample of the cell
    int *new_d = name + K;                         // [K] slot inside the row
    int *rname = new_d + K;                        // [R]
    int *new_r = rname + R;                        // [R]
    int *ccount = new_r + R;                       // [K + 1]
    int *rcount = ccount + K + 1;                  // [R + 1]
    int *ng = rcount + R + 1;                      // [G] slots per shard
    __shared__ u64 hsum;
    __shared__ i64 pcs, prs;
    const int tid = threadIdx.x;
    const int j = blockIdx.x;
    const int *lay = B.lay + (size_t)j * N;
    const char *blob = blobs + (size_t)anc[j] * bl.bytes;
    const int *T = (const int *)(blob + bl.off_T);
    const u64 *Q = (const u64 *)(blob + bl.off_Q);
    const int *W = W_all + (size_t)wloc[j] * dm.RG * dm.LP;

    for (int c = tid; c < K; c += SEL_THREADS) name[c] = N;
    for (int c = tid; c <= K; c += SEL_THREADS) ccount[c] = 0;
    for (int r = tid; r <= R; r += SEL_THREADS) rcount[r] = 0;
    for (int r = tid; r < R; r += SEL_THREADS) rname[r] = N;
    for (int g = tid; g < G; g += SEL_THREADS) ng[g] = 0;
    for (int x = tid; x < n_proj * R; x += SEL_THREADS) ph[x] = 0;
    if (tid == 0) { hsum = 0; pcs = 0; prs = 0; }
    __syncthreads();
    for (int i = tid; i < N; i += SEL_THREADS) {
        const int c = lay[i];
        atomicMin(&name[c], i);
        atomicAdd(&ccount[c + 1], 1);
        atomicAdd(&rcount[c / D + 1], 1);
    }
    for (int d = tid; d < D; d += SEL_THREADS) atomicAdd(&ng[g_of_cell[d]], 1);
    __syncthreads();
    for (int c = tid; c < K; c += SEL_THREADS) atomicMin(&rname[c / D], name[c]);
    {   // pairs together, from the group sizes
        i64 a = 0, b = 0;
        for (int c = tid; c < K; c += SEL_THREADS) { const i64 n = ccount[c + 1]; a += n * (n - 1) / 2; }
        for (int r = tid; r < R; r += SEL_THREADS) { const i64 n = rcount[r + 1]; b += n * (n - 1) / 2; }
        if (a) atomicAdd((u64 *)&pcs, (u64)a);
        if (b) atomicAdd((u64 *)&prs, (u64)b);
    }
    __syncthreads();
    // position of every cell among the cells of its shard in its row, and of every row
    for (int c = tid; c < K; c += SEL_THREADS) {
        const int r = c / D, g = g_of_cell[c];
        int pos = 0;
        for (int d2 = 0; d2 < D; ++d2) pos += (g_of_cell[r * D + d2] == g && name[r * D + d2] < name[c]);
        int seen = 0, target = -1;
        for (int d2 = 0; d2 < D && target < 0; ++d2)
            if (g_of_cell[d2] == g) { if (seen == pos) target = d2; ++seen; }
        new_d[c] = target;
    }
    for (int r = tid; r < R; r += SEL_THREADS) {
        int pos = 0;
        for (int r2 = 0; r2 < R; ++r2) pos += (rname[r2] < rname[r]);
        new_r[r] = pos;
    }
    if (tid == 0) {              // exclusive starts of the groups
        int run = 0;
        for (int c = 0; c <= K; ++c) { run += ccount[c]; ccount[c] = run; }
        run = 0;
        for (int r = 0; r <= R; ++r) { run += rcount[r]; rcount[r] = run; }
    }
    __syncthreads();
    for (int c = tid; c <= K; c += SEL_THREADS) B.cstart[(size_t)j * (K + 1) + c] = ccount[c];
    for (int r = tid; r <= R; r += SEL_THREADS) B.rstart[(size_t)j * (R + 1) + r] = rcount[r];
    {
        u64 h = 0;
        for (int i = tid; i < N; i += SEL_THREADS) {
            const int c = lay[i];
            const int cn = new_r[c / D] * D + new_d[c];
            B.canon[(size_t)j * N + i] = cn;
            h += sel_mix((u64)i * (u64)K + (u64)cn);
        }
        atomicAdd((unsigned long long *)&hsum, (unsigned long long)h);
    }
    __syncthreads();
    // group lists (order inside a group does not matter to the pair counts)
    for (int i = tid; i < N; i += SEL_THREADS) {
        const int c = lay[i];
        B.clist[(size_t)j * N + atomicAdd(&ccount[c], 1)] = i;
        B.rlist[(size_t)j * N + atomicAdd(&rcount[c / D], 1)] = i;
    }
    // row features -> projections
    const i64 CD = (i64)dm.C * D;
    for (int x = tid; x < R * F; x += SEL_THREADS) {
        const int r = x / F, f = x % F;
        i64 h;
        if (f < 2) {
            if (f == 0) { i64 s = 0; for (int d = 0; d < D; ++d) s += T[r * D + d]; h = (s << 16) / CD; }
            else { u64 s = 0; for (int d = 0; d < D; ++d) s += Q[r * D + d]; h = (i64)((s << 16) / ((u64)CD * (u64)dm.C)); }
        } else {
            const int g = (f - 2) / L, l = (f - 2) % L;
            const int *wr = W + ((size_t)r * G + g) * dm.LP + (size_t)l * P;
            int m = 0;
            for (int p = 0; p < P; ++p) m = max(m, wr[p]);
            h = ((i64)m << 16) / ((i64)dm.k * dm.C * ng[g]);
        }
        for (int k = 0; k < n_proj; ++k)
            atomicAdd((unsigned long long *)&ph[k * R + r], (unsigned long long)(sgn[k * F + f] ? -h : h));
    }
    __syncthreads();
    for (int x = tid; x < n_proj * R; x += SEL_THREADS) {        // sort each projection by counting
        const int k = x / R, r = x % R;
        const i64 v = ph[x];
        int pos = 0;
        for (int r2 = 0; r2 < R; ++r2) { const i64 o = ph[k * R + r2]; pos += (o < v) || (o == v && r2 < r); }
        B.phi[((size_t)j * n_proj + k) * R + pos] = v;
    }
    if (tid == 0) { B.hash[j] = hsum; B.pc[j] = pcs; B.pr[j] = prs; }
}

// ---- CanonicalMap: is member j the representative of its class? ---------------------------------
__global__ void __launch_bounds__(SEL_THREADS)
k_sel_map(int N, int Ppop, const int *__restrict__ canon, const u64 *__restrict__ hash,
          const i64 *__restrict__ score, int *__restrict__ rep)
{
    __shared__ int beaten;
    const int j = blockIdx.x;
    if (threadIdx.x == 0) beaten = 0;
    __syncthreads();
    const u64 hj = hash[j];
    const i64 a0 = score[3 * (size_t)j], a1 = score[3 * (size_t)j + 1], a2 = score[3 * (size_t)j + 2];
    for (int o = threadIdx.x; o < Ppop; o += SEL_THREADS) {
        if (o == j || hash[o] != hj) continue;
        bool same = true;
        for (int i = 0; i < N && same; ++i) same = canon[(size_t)j * N + i] == canon[(size_t)o * N + i];
        if (!same) continue;
        const i64 b0 = score[3 * (size_t)o], b1 = score[3 * (size_t)o + 1], b2 = score[3 * (size_t)o + 2];
        if (rp_lex_less(b0, b1, b2, a0, a1, a2) || (!rp_lex_less(a0, a1, a2, b0, b1, b2) && o < j)) beaten = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) rep[j] = !beaten;
}

// ---- plan distances between representatives ------------------------------------------------------
// Pairs together in both labelings: every pair of one group of a is looked up in b.
__device__ __forceinline__ i64 sel_both(const int *__restrict__ list, const int *__restrict__ start, int n_groups,
                                        const int *__restrict__ lb, int div_b, int tid)
{
    i64 both = 0;
    for (int g = 0; g < n_groups; ++g) {
        const int s = start[g], n = start[g + 1] - s;
        const int np = n * (n - 1) / 2;
        for (int x = tid; x < np; x += SEL_THREADS) {
            // x-th pair (u < v) of the group
            int v = (int)((1.0f + sqrtf(1.0f + 8.0f * (float)x)) * 0.5f);
            while (v * (v - 1) / 2 > x) --v;
            while ((v + 1) * v / 2 <= x) ++v;
            const int u = x - v * (v - 1) / 2;
            both += (lb[list[s + u]] / div_b == lb[list[s + v]] / div_b);
        }
    }
    return both;
}

__global__ void __launch_bounds__(SEL_THREADS)
k_sel_dist(RpDims dm, int Ppop, int n_proj, const int *__restrict__ rep, SelBuf B, i64 *__restrict__ dist, int cells_by_table)
{
    const int a = blockIdx.x, b = blockIdx.y;
    if (b <= a) { if (a == b && threadIdx.x == 0) dist[(size_t)a * Ppop + a] = 0; return; }
    if (!rep[a] || !rep[b]) return;
    __shared__ i64 acc[3];
    __shared__ int tab[SEL_TABLE];                 // row-by-row contingency counts when R*R fits
    extern __shared__ int ctab[];                  // cell-by-cell contingency counts when K*K ints fit (cells_by_table)
    const int tid = threadIdx.x;
    const int N = dm.N, K = dm.K, R = dm.R, D = dm.D;
    const bool rows_by_table = R * R <= SEL_TABLE;
    if (tid < 3) acc[tid] = 0;
    if (rows_by_table) for (int x = tid; x < R * R; x += SEL_THREADS) tab[x] = 0;
    if (cells_by_table) for (int x = tid; x < K * K; x += SEL_THREADS) ctab[x] = 0;
    __syncthreads();
    const int *la = B.lay + (size_t)a * N, *lb = B.lay + (size_t)b * N;
    i64 bc = 0;
    if (cells_by_table) {
        // pairs in the same cell of both plans = sum over (cell of a, cell of b) of C(count, 2): N counts
        // instead of one look-up per pair of a cell's samples (cells of hundreds of samples)
        for (int i = tid; i < N; i += SEL_THREADS) atomicAdd(&ctab[la[i] * K + lb[i]], 1);
        __syncthreads();
        for (int x = tid; x < K * K; x += SEL_THREADS) { const i64 n = ctab[x]; bc += n * (n - 1) / 2; }
    } else {
        bc = sel_both(B.clist + (size_t)a * N, B.cstart + (size_t)a * (K + 1), K, lb, 1, tid);
    }
    i64 br = 0;
    if (rows_by_table) {
        // pairs in the same row of both plans = sum over (row of a, row of b) of C(count, 2)
        for (int i = tid; i < N; i += SEL_THREADS) atomicAdd(&tab[(la[i] / D) * R + lb[i] / D], 1);
        __syncthreads();
        for (int x = tid; x < R * R; x += SEL_THREADS) { const i64 n = tab[x]; br += n * (n - 1) / 2; }
    } else {
        br = sel_both(B.rlist + (size_t)a * N, B.rstart + (size_t)a * (R + 1), R, lb, D, tid);
    }
    i64 sw = 0;
    const i64 *pa = B.phi + (size_t)a * n_proj * R, *pb = B.phi + (size_t)b * n_proj * R;
    for (int x = tid; x < n_proj * R; x += SEL_THREADS) { const i64 d = pa[x] - pb[x]; sw += d < 0 ? -d : d; }
    for (int o = 16; o; o >>= 1) {
        bc += __shfl_xor_sync(0xffffffffu, bc, o);
        br += __shfl_xor_sync(0xffffffffu, br, o);
        sw += __shfl_xor_sync(0xffffffffu, sw, o);
    }
    if ((tid & 31) == 0) {
        atomicAdd((unsigned long long *)&acc[0], (unsigned long long)bc);
        atomicAdd((unsigned long long *)&acc[1], (unsigned long long)br);
        atomicAdd((unsigned long long *)&acc[2], (unsigned long long)sw);
    }
    __syncthreads();
    if (tid == 0) {
        const int F = 2 + dm.G * dm.L;
        const i64 uc = B.pc[a] + B.pc[b] - acc[0], ur = B.pr[a] + B.pr[b] - acc[1];
        i64 d = 0;
        if (uc) d += ((i64)1 << 20) - (acc[0] << 20) / uc;
        if (ur) d += ((i64)1 << 20) - (acc[1] << 20) / ur;
        d += (acc[2] * 16) / ((i64)n_proj * R * F);
        dist[(size_t)a * Ppop + b] = d;
        dist[(size_t)b * Ppop + a] = d;
    }
}

// ---- greedy selection (one CTA) -------------------------------------------------------------------
#define GREEDY_THREADS 1024
struct SelPick { i64 v0, v1, v2; int j; };

__global__ void __launch_bounds__(GREEDY_THREADS)
k_sel_greedy(int Ppop, const int *__restrict__ rep, const i64 *__restrict__ score, const i64 *__restrict__ dist,
             i64 eta_q16, i64 *__restrict__ mind, i64 *__restrict__ pen, int *__restrict__ order, int *__restrict__ n_distinct)
{
    __shared__ SelPick red[GREEDY_THREADS / 32];
    __shared__ SelPick pick_s;
    __shared__ int nd_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) nd_s = 0;
    __syncthreads();
    // winner by score (lowest triple, lowest index) and the number of representatives
    SelPick best = { 0x7fffffffffffffffll, 0x7fffffffffffffffll, 0x7fffffffffffffffll, 0x7fffffff };
    int cnt = 0;
    for (int j = tid; j < Ppop; j += GREEDY_THREADS) {
        if (!rep[j]) continue;
        ++cnt;
        const i64 s0 = score[3 * (size_t)j], s1 = score[3 * (size_t)j + 1], s2 = score[3 * (size_t)j + 2];
        if (rp_lex_less(s0, s1, s2, best.v0, best.v1, best.v2)) { best.v0 = s0; best.v1 = s1; best.v2 = s2; best.j = j; }
    }
    if (cnt) atomicAdd(&nd_s, cnt);
    auto reduce_min = [&](SelPick b) {
        for (int o = 16; o; o >>= 1) {
            SelPick ot;
            ot.v0 = __shfl_xor_sync(0xffffffffu, b.v0, o); ot.v1 = __shfl_xor_sync(0xffffffffu, b.v1, o);
            ot.v2 = __shfl_xor_sync(0xffffffffu, b.v2, o); ot.j = __shfl_xor_sync(0xffffffffu, b.j, o);
            if (rp_lex_less(ot.v0, ot.v1, ot.v2, b.v0, b.v1, b.v2) ||
                (ot.v0 == b.v0 && ot.v1 == b.v1 && ot.v2 == b.v2 && ot.j < b.j)) b = ot;
        }
        if (lane == 0) red[warp] = b;
        __syncthreads();
        if (tid == 0) {
            for (int w = 1; w < GREEDY_THREADS / 32; ++w) {
                const SelPick ot = red[w];
                if (rp_lex_less(ot.v0, ot.v1, ot.v2, b.v0, b.v1, b.v2) ||
                    (ot.v0 == b.v0 && ot.v1 == b.v1 && ot.v2 == b.v2 && ot.j < b.j)) b = ot;
            }
            pick_s = b;
        }
        __syncthreads();
    };
    reduce_min(best);
    const int nd = nd_s;
    const i64 s0 = pick_s.v0;
    int last = pick_s.j;
    for (int j = tid; j < Ppop; j += GREEDY_THREADS) {
        i64 p = 0;
        if (rep[j] && s0 > 0) {
            const unsigned __int128 gap = ((unsigned __int128)(u64)(score[3 * (size_t)j] - s0) << 20) / (u64)s0;
            p = (i64)((gap * (unsigned __int128)(u64)eta_q16) >> 16);
        }
        pen[j] = p;
        mind[j] = rep[j] ? 0x7fffffffffffffffll : -1;      // -1 = not a candidate (or already selected)
    }
    __syncthreads();
    for (int n = 0; n < nd; ++n) {
        if (tid == 0) order[n] = last;
        // negated objective so that the same lexicographic minimum applies: maximise v, lowest index
        SelPick b = { 0x7fffffffffffffffll, 0, 0, 0x7fffffff };
        for (int j = tid; j < Ppop; j += GREEDY_THREADS) {
            if (j == last) mind[j] = -1;
            i64 m = mind[j];
            if (m < 0) continue;
            const i64 d = dist[(size_t)j * Ppop + last];
            if (d < m) { m = d; mind[j] = m; }
            const i64 neg = -(m - pen[j]);
            if (neg < b.v0 || (neg == b.v0 && j < b.j)) { b.v0 = neg; b.j = j; }
        }
        reduce_min(b);
        last = pick_s.j;
    }
    for (int m = nd + tid; m < Ppop; m += GREEDY_THREADS) order[m] = order[m % nd];
    if (tid == 0) *n_distinct = nd;
}

__global__ void k_sel_fill(int N, const int *__restrict__ order, const int *__restrict__ lay, int *__restrict__ out)
{
    const int m = blockIdx.x;
    const int *src = lay + (size_t)order[m] * N;
    for (int i = threadIdx.x; i < N; i += blockDim.x) out[(size_t)m * N + i] = src[i];
}

// lay [P][N]: the population's layouts (input); out [P][N]: the selected population.
// score [P][3]: exact scores of the members.  order [P], n_distinct [1], dist [P][P] device outputs.
int rp_launch_select(rp_ctx *c, int *lay, int *out, const i64 *score, int n_proj, i64 eta_q16, int *order,
                     int *n_distinct, i64 *dist)
{
    const RpDims &dm = c->dm;
    const size_t P = (size_t)c->Ppop;
    const int F = 2 + dm.G * dm.L;
    SelBuf B;
    B.lay = lay;
    unsigned char *sgn = nullptr;
    int *rep = nullptr;
    i64 *mind = nullptr, *pen = nullptr;
    B.canon = nullptr; B.hash = nullptr; B.clist = nullptr; B.cstart = nullptr; B.rlist = nullptr; B.rstart = nullptr;
    B.pc = nullptr; B.pr = nullptr; B.phi = nullptr;
    int st = dev_alloc(c, &B.canon, P * dm.N);
    if (st == RP_OK) st = dev_alloc(c, &B.hash, P);
    if (st == RP_OK) st = dev_alloc(c, &B.clist, P * dm.N);
    if (st == RP_OK) st = dev_alloc(c, &B.cstart, P * (dm.K + 1));
    if (st == RP_OK) st = dev_alloc(c, &B.rlist, P * dm.N);
    if (st == RP_OK) st = dev_alloc(c, &B.rstart, P * (dm.R + 1));
    if (st == RP_OK) st = dev_alloc(c, &B.pc, P);
    if (st == RP_OK) st = dev_alloc(c, &B.pr, P);
    if (st == RP_OK) st = dev_alloc(c, &B.phi, P * n_proj * dm.R);
    if (st == RP_OK) st = dev_alloc(c, &sgn, (size_t)F * n_proj);
    if (st == RP_OK) st = dev_alloc(c, &rep, P);
    if (st == RP_OK) st = dev_alloc(c, &mind, P);
    if (st == RP_OK) st = dev_alloc(c, &pen, P);
    const size_t smem = sizeof(i64) * (size_t)n_proj * dm.R + sizeof(int) * ((size_t)3 * dm.K + 3 * dm.R + dm.G + 2) + 16;
    if (st == RP_OK && smem > 200 * 1024) st = RP_ERR_RANGE;
    cudaError_t e = cudaSuccess;
    if (st == RP_OK) {
        if (smem > 32 * 1024) e = cudaFuncSetAttribute(k_sel_prepare, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) {
            k_sel_signs<<<(F * n_proj + 255) / 256, 256, 0, c->stream>>>(F, n_proj, (u32)c->cfg.seed, (u32)(c->cfg.seed >> 32), sgn);
            k_sel_prepare<<<(int)P, SEL_THREADS, smem, c->stream>>>(dm, c->bl, c->buf[c->cur].blob, c->d_anc, c->d_W, c->d_wloc,
                                                                    (const unsigned short *)(c->d_static + c->sl.off_g), sgn, n_proj, B);
            k_sel_map<<<(int)P, SEL_THREADS, 0, c->stream>>>(dm.N, (int)P, B.canon, B.hash, score, rep);
            e = cudaMemsetAsync(dist, 0, sizeof(i64) * P * P, c->stream);
        }
        if (e == cudaSuccess) {
            // cell-by-cell counts in shared memory where they fit twice per SM beside the row table
            const size_t ctab_bytes = sizeof(int) * (size_t)dm.K * dm.K;
            const int cells_by_table = ctab_bytes <= 80 * 1024;
            if (cells_by_table && ctab_bytes > 24 * 1024)
                e = cudaFuncSetAttribute(k_sel_dist, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
            if (e == cudaSuccess)
                k_sel_dist<<<dim3((unsigned)P, (unsigned)P), SEL_THREADS, cells_by_table ? ctab_bytes : 0, c->stream>>>(
                    dm, (int)P, n_proj, rep, B, dist, cells_by_table);
            k_sel_greedy<<<1, GREEDY_THREADS, 0, c->stream>>>((int)P, rep, score, dist, eta_q16, mind, pen, order, n_distinct);
            k_sel_fill<<<(int)P, 256, 0, c->stream>>>(dm.N, order, lay, out);
            g_rp_launches += 6;
            e = cudaGetLastError();
        }
    }
    dev_free(c, B.canon); dev_free(c, B.hash); dev_free(c, B.clist); dev_free(c, B.cstart); dev_free(c, B.rlist);
    dev_free(c, B.rstart); dev_free(c, B.pc); dev_free(c, B.pr); dev_free(c, B.phi); dev_free(c, sgn); dev_free(c, rep);
    dev_free(c, mind); dev_free(c, pen);
    if (e != cudaSuccess) { g_rp_last_cuda_error = (int)e; return RP_ERR_CUDA; }
    return st;
}
