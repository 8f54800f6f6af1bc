/*
 * RoutePack planner -- plain CPU oracle (TEST INFRASTRUCTURE, not the product).
 *
 * A slow, direct restatement of what the planner's hot path computes, written from the
 * paper's problem formulation (Section 3) and solver description (Section 4.1).  It is
 * the checker the CUDA library is compared against; it shares no code, header, table or
 * helper with that library, and the library never calls it.  Only tests, the smoke
 * check and the benchmark's CPU-baseline leg may build or load this file.
 *
 * Every decision the search takes (feasibility, score order, Metropolis accept,
 * resampling ancestors) is taken on integers, so a second implementation can reproduce
 * the whole trajectory bit for bit.  The paper states the objective on real numbers;
 * the integer form used here is the same objective multiplied by SC = 2^8 * C^2
 * (C = token cap), which makes every term an exact integer:
 *
 *   cell statistics (Eq. cell-token-statistics):  T = sum t_i,  Q = sum t_i^2
 *   attention       (Eq. stage-aware-attention):  Afx[r][g] = sum_s max_{d in D_g}
 *                                                   (ahat_s*C*T[r][d] + bhat_s*Q[r][d])
 *   rank load       (Eq. row-expert-load):        W[r][g][l][p] = sum_{d in D_g} sum_{i in cell} q[i][l][p]
 *   expert cost     (Eq. row-expert-cost):        Efx[r][g] = 2^8*C * sum_l max_p W[r][g][l][p]
 *   row cost, shard work:                         Jfx = Afx + Efx,  U[g] = sum_r Jfx[r][g]
 *   score           (Eq. lexicographic-score):    (max_g U, sum_g U, max_{r,g} Jfx), lexicographic
 *   energy          (Eq. pa-energy):              Efx_scalar = s0 + floor(s1/10^6) + floor(s2/10^9)
 *
 * with ahat_s = round(alpha_s * 2^8), bhat_s = round(beta_s * 2^8).  orc_eval_f64 below
 * evaluates the paper's real-valued formulas directly, to show the two agree.
 *
 * Parity status of the pieces the paper leaves open (values it never prints): the law
 * of the guided-proposal bias (a tournament of two here), the attention coefficients, the
 * temperature schedule, the relocation probability and the FixedRowFFD details are
 * "parity unpinned" against the paper; they are fixed by the readings listed beside each
 * function.  What the paper does fix about GuidedProposal (p_guide = 0.8, sources biased
 * to a large J, targets to a small one, the attention straggler in proportion to its
 * contribution, the other branch uniform) and the energy coefficients of Eq. pa-energy
 * are pinned through orc_propose_once / orc_energy at the end of this file.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

typedef unsigned __int128 u128;

#define ORC_FBITS 8          /* fixed-point fraction bits of the attention coefficients */
#define ORC_MAX_STAGES 8

/* ------------------------------------------------------------------------------------ */
/* Counter-based random numbers: Philox4x32 with 10 rounds (Salmon et al., SC'11).      */
/* Used for every random draw of Algorithm 3 so that streams can be re-created exactly. */
/* ------------------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Stream layout: counter = (step k, level n, chain slot j, purpose), key = 64-bit seed. */
enum { ORC_DRAW_A = 0, ORC_DRAW_B = 1, ORC_DRAW_ACCEPT = 2, ORC_DRAW_RESAMPLE = 3 };

static void draw(uint64_t seed, uint32_t step, uint32_t level, uint32_t slot, uint32_t purpose,
                 uint32_t out[4])
{
    uint32_t ctr[4] = { step, level, slot, purpose };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    orc_philox4x32_10(ctr, key, out);
}

/* Uniform index in [0, n) from a 32-bit word: floor(x * n / 2^32). */
static inline int32_t pick(uint32_t x, int32_t n)
{
    return (int32_t)(((uint64_t)x * (uint64_t)(uint32_t)n) >> 32);
}

/* ------------------------------------------------------------------------------------ */
/* Integer transcendental functions used by the Metropolis test and the Boltzmann       */
/* weights of Algorithm 3 (the paper writes exp(); decisions here need exact bits).     */
/* ------------------------------------------------------------------------------------ */

/* -log2(u) for u = (x+1)/2^32 in (0,1], as an unsigned Q32 number (32 fraction bits).
 * log2(x+1) = e + log2(m), m in [1,2): the 24 leading fraction bits of log2(m) come from
 * the textbook square-and-compare recurrence on m held with 63 fraction bits; products
 * are truncated.  The low 8 fraction bits of the result are zero. */
uint64_t orc_nl2(uint32_t x)
{
    uint64_t v = (uint64_t)x + 1u;              /* 1 .. 2^32 */
    int e = 63 - __builtin_clzll(v);            /* floor(log2 v), 0 .. 32 */
    uint64_t m = v << (63 - e);                 /* m / 2^63 in [1,2) */
    uint64_t frac = 0;
    for (int i = 0; i < 24; ++i) {
        uint64_t sq = (uint64_t)(((u128)m * m) >> 64);   /* m^2 with 62 fraction bits, in [1,4) */
        if (sq >> 63) { frac = (frac << 1) | 1u; m = sq; }        /* >= 2: bit is 1, halve */
        else          { frac = (frac << 1);      m = sq << 1; }
    }
    return ((uint64_t)(32 - e) << 32) - (frac << 8);
}

/* floor(2^63 * 2^(-2^-i)), i = 1..24.  Written by oracle/gen_exp2_table.py from
 * 80-digit decimal arithmetic; the tests recompute them the same way and compare. */
static const uint64_t ORC_EXP2_STEP[24] = {
    0x5A827999FCEF3242ull, 0x6BA27E656B4EB57Aull, 0x75606373EE921C97ull, 0x7A92BE8A92436616ull,
    0x7D41D96DB915019Dull, 0x7E9F06067A4360BAull, 0x7F4F08AE3DC7C425ull, 0x7FA765ACA88F6452ull,
    0x7FD3AB290E46D768ull, 0x7FE9D3A8E07BF085ull, 0x7FF4E9597BED93AAull, 0x7FFA748DFF8DC61Eull,
    0x7FFD3A3F50020332ull, 0x7FFE9D1DBC0A75A9ull, 0x7FFF4E8E6306ED58ull, 0x7FFFA74712C3CDFDull,
    0x7FFFD3A381B1FA28ull, 0x7FFFE9D1BEED0189ull, 0x7FFFF4E8DEFB81D7ull, 0x7FFFFA746F5F012Full,
    0x7FFFFD3A37A7D0A8ull, 0x7FFFFE9D1BD1FC58ull, 0x7FFFFF4E8DE8832Dull, 0x7FFFFFA746F422D6ull,
};
void orc_exp2_table(uint64_t tab[24]) { memcpy(tab, ORC_EXP2_STEP, sizeof ORC_EXP2_STEP); }

/* 2^(-z) for unsigned Q32 z, returned in Q32 (2^32 = 1.0).  Only the 24 leading fraction
 * bits of z are used; z >= 32 gives 0. */
uint64_t orc_exp2neg(uint64_t z)
{
    const uint64_t *tab = ORC_EXP2_STEP;
    uint64_t ip = z >> 32;
    if (ip >= 32) return 0;
    uint64_t acc = 1ull << 63;                               /* 1.0 with 63 fraction bits */
    for (int i = 1; i <= 24; ++i)
        if ((z >> (32 - i)) & 1u)
            acc = (uint64_t)(((u128)acc * tab[i - 1]) >> 63);
    return (acc >> 31) >> ip;
}

/* ------------------------------------------------------------------------------------ */
/* Input checks (Section 3.1): 1 <= t_i <= C, a >= 0, sum_e a[i][l][e] = k * t_i.       */
/* Returns 0 when the window is consistent, else 1 + index of the first bad sample.     */
/* ------------------------------------------------------------------------------------ */
int64_t orc_check_window(int32_t N, int32_t L, int32_t E, int32_t k, int32_t C,
                         const int32_t *t, const int32_t *a)
{
    for (int32_t i = 0; i < N; ++i) {
        if (t[i] < 1 || t[i] > C) return 1 + (int64_t)i;
        for (int32_t l = 0; l < L; ++l) {
            int64_t s = 0;
            for (int32_t e = 0; e < E; ++e) {
                int32_t v = a[((size_t)i * L + l) * E + e];
                if (v < 0) return 1 + (int64_t)i;
                s += v;
            }
            if (s != (int64_t)k * t[i]) return 1 + (int64_t)i;
        }
    }
    return 0;
}

/* Aggregate expert load of the optimizer window (Section 3.3): Lagg[l][e] = sum_i a[i][l][e]. */
void orc_aggregate(int32_t N, int32_t L, int32_t E, const int32_t *a, int64_t *Lagg)
{
    memset(Lagg, 0, sizeof(int64_t) * (size_t)L * E);
    for (int32_t i = 0; i < N; ++i)
        for (int32_t l = 0; l < L; ++l)
            for (int32_t e = 0; e < E; ++e)
                Lagg[(size_t)l * E + e] += a[((size_t)i * L + l) * E + e];
}

/* Layer-local LPT placement (Algorithm 1) for one layer.
 * Experts are visited by decreasing load, ties by expert id; each goes to the rank with
 * the smallest current load among ranks that still have a free slot, ties by rank id.
 * Reading of slot(p, n): slots are numbered rank-major, slot = p*H + n (n counted from 0),
 * so owner(v) = v / H.  pi[e] = slot, Gload[p] = final aggregate load of rank p. */
void orc_lpt_layer(int32_t E, int32_t P, const int64_t *Le, int32_t *pi, int64_t *Gload)
{
    int32_t H = E / P;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * E);
    int32_t *nslots = (int32_t *)calloc(P, sizeof(int32_t));
    for (int32_t p = 0; p < P; ++p) Gload[p] = 0;
    for (int32_t e = 0; e < E; ++e) order[e] = e;
    /* insertion sort by (-load, id): plain and stable */
    for (int32_t x = 1; x < E; ++x) {
        int32_t e = order[x], y = x;
        while (y > 0 && (Le[order[y - 1]] < Le[e] ||
                         (Le[order[y - 1]] == Le[e] && order[y - 1] > e))) {
            order[y] = order[y - 1];
            --y;
        }
        order[y] = e;
    }
    for (int32_t x = 0; x < E; ++x) {
        int32_t e = order[x], best = -1;
        for (int32_t p = 0; p < P; ++p) {
            if (nslots[p] >= H) continue;
            if (best < 0 || Gload[p] < Gload[best]) best = p;
        }
        pi[e] = best * H + nslots[best];
        Gload[best] += Le[e];
        nslots[best] += 1;
    }
    free(order);
    free(nslots);
}

/* Physical-rank demand of every sample (Eq. physical-rank-demand):
 * q[i][l][p] = sum of a[i][l][e] over experts e whose slot pi[l][e] is owned by rank p. */
void orc_project(int32_t N, int32_t L, int32_t E, int32_t P, const int32_t *a,
                 const int32_t *pi, int32_t *q)
{
    int32_t H = E / P;
    memset(q, 0, sizeof(int32_t) * (size_t)N * L * P);
    for (int32_t i = 0; i < N; ++i)
        for (int32_t l = 0; l < L; ++l)
            for (int32_t e = 0; e < E; ++e) {
                int32_t owner = pi[(size_t)l * E + e] / H;
                q[((size_t)i * L + l) * P + owner] += a[((size_t)i * L + l) * E + e];
            }
}

/* ------------------------------------------------------------------------------------ */
/* Row count and length-only seed (Section 3.2; Algorithm 2, first line).               */
/* Reading (the paper names a "fixed-bin feasibility check" and FixedRowFFD without     */
/* details): try R = R_lb, R_lb+1, ... with R_lb = max(1, min_rows, ceil(sum t/(C*D))); */
/* for each R run first-fit-decreasing into K = R*D bins: samples in order (-t_i, i),   */
/* the K longest open bins 0..K-1 (so no cell is empty), every later sample goes to the */
/* lowest-numbered bin it fits in.  The first R that packs is R*; it is certified       */
/* minimal when R* == R_lb (a true lower bound).  Bin b is cell (row b / D, slot b % D).*/
/* Returns R* (>0), or 0 when no R <= N/D packs (or some t_i > C, or N < D).            */
/* ------------------------------------------------------------------------------------ */
int32_t orc_pack_ffd(int32_t N, int32_t C, int32_t D, int32_t min_rows, const int32_t *t,
                     int32_t *cell_of, int32_t *certified)
{
    *certified = 0;
    if (N < D) return 0;
    int64_t total = 0;
    for (int32_t i = 0; i < N; ++i) { if (t[i] > C || t[i] < 1) return 0; total += t[i]; }
    int64_t capRow = (int64_t)C * D;
    int64_t Rlb = (total + capRow - 1) / capRow;
    if (Rlb < 1) Rlb = 1;
    if (Rlb < min_rows) Rlb = min_rows;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * N);
    for (int32_t i = 0; i < N; ++i) order[i] = i;
    for (int32_t x = 1; x < N; ++x) {               /* insertion sort by (-t, i) */
        int32_t s = order[x], y = x;
        while (y > 0 && (t[order[y - 1]] < t[s] || (t[order[y - 1]] == t[s] && order[y - 1] > s))) {
            order[y] = order[y - 1];
            --y;
        }
        order[y] = s;
    }
    int32_t Rstar = 0;
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * (size_t)N);
    for (int64_t R = Rlb; R * D <= N && !Rstar; ++R) {
        int32_t K = (int32_t)(R * D);
        int ok = 1;
        for (int32_t b = 0; b < K; ++b) fill[b] = 0;
        for (int32_t x = 0; x < N && ok; ++x) {
            int32_t s = order[x], b;
            if (x < K) b = x;
            else {
                for (b = 0; b < K; ++b) if (fill[b] + t[s] <= C) break;
                if (b == K) { ok = 0; break; }
            }
            fill[b] += t[s];
            cell_of[s] = b;
        }
        if (ok) { Rstar = (int32_t)R; *certified = (R == Rlb); }
    }
    free(order);
    free(fill);
    return Rstar;
}

/* ------------------------------------------------------------------------------------ */
/* Problem description shared by scoring and annealing.                                  */
/* ------------------------------------------------------------------------------------ */
typedef struct {
    int32_t N, L, P, D, G, R, S;      /* samples, MoE layers, EP ranks, DP slots, EDP shards, rows, stages */
    int32_t C;                        /* token cap */
    const int32_t *edp_of_dp;         /* [D] -> shard g */
    int64_t ahat[ORC_MAX_STAGES];     /* round(alpha_s * 2^8) */
    int64_t bhat[ORC_MAX_STAGES];     /* round(beta_s  * 2^8) */
    const int32_t *t;                 /* [N] */
    const int32_t *q;                 /* [N][L][P] */
} orc_problem;

typedef struct {                      /* one layout and everything cached about it */
    int32_t *cell_of;                 /* [N]  cell = r*D + d */
    int64_t *T, *Q;                   /* [R*D] */
    int32_t *cnt;                     /* [R*D] */
    int32_t *W;                       /* [R][G][L][P] */
    int64_t *Afx, *Efx;               /* [R][G] */
    int64_t *U;                       /* [G] */
    int64_t s[3];
} orc_state;

static void fill_problem(orc_problem *pb, int32_t N, int32_t L, int32_t P, int32_t D, int32_t G,
                         int32_t R, int32_t C, const int32_t *edp_of_dp, int32_t S,
                         const double *alpha, const double *beta, const int32_t *t, const int32_t *q)
{
    pb->N = N; pb->L = L; pb->P = P; pb->D = D; pb->G = G; pb->R = R; pb->S = S; pb->C = C;
    pb->edp_of_dp = edp_of_dp; pb->t = t; pb->q = q;
    for (int32_t s = 0; s < S; ++s) {
        pb->ahat[s] = (int64_t)floor(alpha[s] * (double)(1 << ORC_FBITS) + 0.5);
        pb->bhat[s] = (int64_t)floor(beta[s] * (double)(1 << ORC_FBITS) + 0.5);
    }
}

static orc_state *state_new(const orc_problem *pb)
{
    orc_state *st = (orc_state *)calloc(1, sizeof *st);
    size_t K = (size_t)pb->R * pb->D, RG = (size_t)pb->R * pb->G;
    st->cell_of = (int32_t *)calloc(pb->N, sizeof(int32_t));
    st->T = (int64_t *)calloc(K, sizeof(int64_t));
    st->Q = (int64_t *)calloc(K, sizeof(int64_t));
    st->cnt = (int32_t *)calloc(K, sizeof(int32_t));
    st->W = (int32_t *)calloc(RG * pb->L * pb->P, sizeof(int32_t));
    st->Afx = (int64_t *)calloc(RG, sizeof(int64_t));
    st->Efx = (int64_t *)calloc(RG, sizeof(int64_t));
    st->U = (int64_t *)calloc(pb->G, sizeof(int64_t));
    return st;
}
static void state_free(orc_state *st)
{
    if (!st) return;
    free(st->cell_of); free(st->T); free(st->Q); free(st->cnt);
    free(st->W); free(st->Afx); free(st->Efx); free(st->U); free(st);
}
static void state_copy(const orc_problem *pb, orc_state *dst, const orc_state *src)
{
    size_t K = (size_t)pb->R * pb->D, RG = (size_t)pb->R * pb->G;
    memcpy(dst->cell_of, src->cell_of, sizeof(int32_t) * pb->N);
    memcpy(dst->T, src->T, sizeof(int64_t) * K);
    memcpy(dst->Q, src->Q, sizeof(int64_t) * K);
    memcpy(dst->cnt, src->cnt, sizeof(int32_t) * K);
    memcpy(dst->W, src->W, sizeof(int32_t) * RG * pb->L * pb->P);
    memcpy(dst->Afx, src->Afx, sizeof(int64_t) * RG);
    memcpy(dst->Efx, src->Efx, sizeof(int64_t) * RG);
    memcpy(dst->U, src->U, sizeof(int64_t) * pb->G);
    memcpy(dst->s, src->s, sizeof dst->s);
}

/* A remembered layout: the assignment and its score (enough to name a plan). */
typedef struct { int32_t *cell_of; int64_t s[3]; } orc_plan;
static orc_plan *plan_new(const orc_problem *pb)
{
    orc_plan *pl = (orc_plan *)calloc(1, sizeof *pl);
    pl->cell_of = (int32_t *)calloc(pb->N, sizeof(int32_t));
    return pl;
}
static void plan_free(orc_plan *pl) { if (pl) { free(pl->cell_of); free(pl); } }
static void plan_take(const orc_problem *pb, orc_plan *dst, const int32_t *cell_of, const int64_t s[3])
{
    memcpy(dst->cell_of, cell_of, sizeof(int32_t) * pb->N);
    memcpy(dst->s, s, sizeof dst->s);
}

/* Attention cost of row r on shard g from the cell statistics (Eq. stage-aware-attention):
 * within a cell the linear and pair terms are added first, the maximum over the shard's
 * DP slots is taken per stage, and stages are summed afterwards. */
static int64_t attention_fx(const orc_problem *pb, const orc_state *st, int32_t r, int32_t g)
{
    int64_t sum = 0;
    for (int32_t s = 0; s < pb->S; ++s) {
        int64_t worst = 0;
        for (int32_t d = 0; d < pb->D; ++d) {
            if (pb->edp_of_dp[d] != g) continue;
            size_t c = (size_t)r * pb->D + d;
            int64_t v = pb->ahat[s] * pb->C * st->T[c] + pb->bhat[s] * st->Q[c];
            if (v > worst) worst = v;
        }
        sum += worst;
    }
    return sum;
}

/* Expert cost of row r on shard g (Eq. row-expert-cost): busiest rank per layer, summed. */
static int64_t expert_fx(const orc_problem *pb, const orc_state *st, int32_t r, int32_t g)
{
    const int32_t *w = st->W + ((size_t)r * pb->G + g) * pb->L * pb->P;
    int64_t sum = 0;
    for (int32_t l = 0; l < pb->L; ++l) {
        int32_t worst = 0;
        for (int32_t p = 0; p < pb->P; ++p)
            if (w[(size_t)l * pb->P + p] > worst) worst = w[(size_t)l * pb->P + p];
        sum += worst;
    }
    return sum * ((int64_t)pb->C << ORC_FBITS);
}

/* Shard work and the score tuple (Eq. lexicographic-score) from the cached row costs. */
static void rescore_from_rows(const orc_problem *pb, orc_state *st)
{
    int64_t s0 = 0, s1 = 0, s2 = 0;
    for (int32_t g = 0; g < pb->G; ++g) st->U[g] = 0;
    for (int32_t r = 0; r < pb->R; ++r)
        for (int32_t g = 0; g < pb->G; ++g) {
            int64_t J = st->Afx[(size_t)r * pb->G + g] + st->Efx[(size_t)r * pb->G + g];
            st->U[g] += J;
            if (J > s2) s2 = J;
        }
    for (int32_t g = 0; g < pb->G; ++g) { s1 += st->U[g]; if (st->U[g] > s0) s0 = st->U[g]; }
    st->s[0] = s0; st->s[1] = s1; st->s[2] = s2;
}

/* Full evaluation of a layout from its sample->cell assignment (Section 3.4). */
static void evaluate(const orc_problem *pb, orc_state *st)
{
    size_t K = (size_t)pb->R * pb->D, RG = (size_t)pb->R * pb->G, LP = (size_t)pb->L * pb->P;
    memset(st->T, 0, sizeof(int64_t) * K);
    memset(st->Q, 0, sizeof(int64_t) * K);
    memset(st->cnt, 0, sizeof(int32_t) * K);
    memset(st->W, 0, sizeof(int32_t) * RG * LP);
    for (int32_t i = 0; i < pb->N; ++i) {
        int32_t c = st->cell_of[i], r = c / pb->D, g = pb->edp_of_dp[c % pb->D];
        st->T[c] += pb->t[i];
        st->Q[c] += (int64_t)pb->t[i] * pb->t[i];
        st->cnt[c] += 1;
        int32_t *w = st->W + ((size_t)r * pb->G + g) * LP;
        const int32_t *qi = pb->q + (size_t)i * LP;
        for (size_t x = 0; x < LP; ++x) w[x] += qi[x];
    }
    for (int32_t r = 0; r < pb->R; ++r)
        for (int32_t g = 0; g < pb->G; ++g) {
            st->Afx[(size_t)r * pb->G + g] = attention_fx(pb, st, r, g);
            st->Efx[(size_t)r * pb->G + g] = expert_fx(pb, st, r, g);
        }
    rescore_from_rows(pb, st);
}

static inline int lex_less(const int64_t a[3], const int64_t b[3])
{
    if (a[0] != b[0]) return a[0] < b[0];
    if (a[1] != b[1]) return a[1] < b[1];
    return a[2] < b[2];
}

/* Scalar search energy (Eq. pa-energy) in the same integer units as the score. */
static inline int64_t energy(const int64_t s[3])
{
    return s[0] + s[1] / 1000000 + s[2] / 1000000000;
}

/* Public: evaluate n layouts.  Outputs are optional (NULL to skip); per layout:
 * T,Q [K], cnt [K], W [R][G][L][P], Afx,Efx [R][G], U [G], score [3]. */
void orc_eval(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C,
              const int32_t *edp_of_dp, int32_t S, const double *alpha, const double *beta,
              const int32_t *t, const int32_t *q, int32_t n_layouts, const int32_t *layouts,
              int64_t *T, int64_t *Q, int32_t *cnt, int32_t *W, int64_t *Afx, int64_t *Efx,
              int64_t *U, int64_t *score)
{
    orc_problem pb;
    fill_problem(&pb, N, L, P, D, G, R, C, edp_of_dp, S, alpha, beta, t, q);
    size_t K = (size_t)R * D, RG = (size_t)R * G, LP = (size_t)L * P;
    orc_state *st = state_new(&pb);
    for (int32_t j = 0; j < n_layouts; ++j) {
        memcpy(st->cell_of, layouts + (size_t)j * N, sizeof(int32_t) * N);
        evaluate(&pb, st);
        if (T) memcpy(T + j * K, st->T, sizeof(int64_t) * K);
        if (Q) memcpy(Q + j * K, st->Q, sizeof(int64_t) * K);
        if (cnt) memcpy(cnt + j * K, st->cnt, sizeof(int32_t) * K);
        if (W) memcpy(W + j * RG * LP, st->W, sizeof(int32_t) * RG * LP);
        if (Afx) memcpy(Afx + j * RG, st->Afx, sizeof(int64_t) * RG);
        if (Efx) memcpy(Efx + j * RG, st->Efx, sizeof(int64_t) * RG);
        if (U) memcpy(U + (size_t)j * G, st->U, sizeof(int64_t) * G);
        if (score) memcpy(score + (size_t)j * 3, st->s, sizeof st->s);
    }
    state_free(st);
}

/* The objective exactly as the paper writes it, on real numbers (Eqs. cell-token-statistics
 * to lexicographic-score), with alpha = ahat/2^8 and beta = bhat/2^8: normalised cell
 * statistics Tbar = sum t/C and Qbar = sum (t/C)^2, A, E = (1/C) sum_l max_p W, J, U. */
void orc_eval_f64(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C,
                  const int32_t *edp_of_dp, int32_t S, const double *alpha, const double *beta,
                  const int32_t *t, const int32_t *q, const int32_t *cell_of, double score[3])
{
    orc_problem pb;
    fill_problem(&pb, N, L, P, D, G, R, C, edp_of_dp, S, alpha, beta, t, q);
    size_t K = (size_t)R * D, LP = (size_t)L * P;
    double *Tb = (double *)calloc(K, sizeof(double)), *Qb = (double *)calloc(K, sizeof(double));
    double *U = (double *)calloc(G, sizeof(double));
    int64_t *w = (int64_t *)malloc(sizeof(int64_t) * LP);
    for (int32_t i = 0; i < N; ++i) {
        double x = (double)t[i] / (double)C;
        Tb[cell_of[i]] += x;
        Qb[cell_of[i]] += x * x;
    }
    double s2 = 0.0;
    for (int32_t r = 0; r < R; ++r)
        for (int32_t g = 0; g < G; ++g) {
            double A = 0.0;
            for (int32_t s = 0; s < S; ++s) {
                double worst = 0.0;
                for (int32_t d = 0; d < D; ++d) {
                    if (edp_of_dp[d] != g) continue;
                    double a_s = (double)pb.ahat[s] / 256.0, b_s = (double)pb.bhat[s] / 256.0;
                    double v = a_s * Tb[(size_t)r * D + d] + b_s * Qb[(size_t)r * D + d];
                    if (v > worst) worst = v;
                }
                A += worst;
            }
            memset(w, 0, sizeof(int64_t) * LP);
            for (int32_t i = 0; i < N; ++i) {
                int32_t c = cell_of[i];
                if (c / D != r || edp_of_dp[c % D] != g) continue;
                for (size_t x = 0; x < LP; ++x) w[x] += q[(size_t)i * LP + x];
            }
            double E = 0.0;
            for (int32_t l = 0; l < L; ++l) {
                int64_t worst = 0;
                for (int32_t p = 0; p < P; ++p) if (w[(size_t)l * P + p] > worst) worst = w[(size_t)l * P + p];
                E += (double)worst;
            }
            E /= (double)C;
            double J = A + E;
            U[g] += J;
            if (J > s2) s2 = J;
        }
    double s0 = 0.0, s1 = 0.0;
    for (int32_t g = 0; g < G; ++g) { s1 += U[g]; if (U[g] > s0) s0 = U[g]; }
    score[0] = s0; score[1] = s1; score[2] = s2;
    free(Tb); free(Qb); free(U); free(w);
}

/* ------------------------------------------------------------------------------------ */
/* One proposal step of a fixed-temperature chain (Algorithm 3, inner loop; Section      */
/* 4.1.2 for GuidedProposal and IncrementalScore).                                       */
/* ------------------------------------------------------------------------------------ */
typedef struct {
    int32_t reloc;      /* 1 = relocation, 0 = swap */
    int32_t i;          /* moved sample */
    int32_t i2;         /* swap partner (swap) */
    int32_t c1, c2;     /* source cell, destination cell */
} orc_move;

static inline int64_t cell_attention_key(const orc_problem *pb, const orc_state *st, int32_t c)
{
    int64_t v = 0;
    for (int32_t s = 0; s < pb->S; ++s)
        v += pb->ahat[s] * pb->C * st->T[c] + pb->bhat[s] * st->Q[c];
    return v;
}
static inline size_t rowshard_of_cell(const orc_problem *pb, int32_t c)
{
    return (size_t)(c / pb->D) * pb->G + pb->edp_of_dp[c % pb->D];
}
static inline int64_t J_of_cell(const orc_problem *pb, const orc_state *st, int32_t c)
{
    size_t rg = rowshard_of_cell(pb, c);
    return st->Afx[rg] + st->Efx[rg];
}

/* GuidedProposal.  Reading of the paper's qualitative description (p_guide = 0.8; source
 * biased to a large J, target to a small one; the attention straggler picked in
 * proportion to its contribution; the other branch uniform):
 *   relocation iff A0 < rho*2^32; guided iff A1 < p_guide*2^32.
 *   uniform branch: sample i = pick(A2,N); partner pick(A3,N) or destination cell pick(A3,K).
 *   guided branch: a tournament of two.  Source candidates pick(A2,N), pick(A3,N).  The
 *   comparison key is the attention cost of the sample's cell with probability Afx/Jfx of
 *   the first candidate's row-shard (test B2*Jfx < Afx*2^32), else the row-shard cost Jfx.
 *   Source = the candidate with the larger key (tie: first).  Target candidates from
 *   B0,B1 (samples for a swap, cells for a relocation); target = smaller key (tie: first).
 * Returns the move; feasibility is decided by the caller. */
static orc_move propose(const orc_problem *pb, const orc_state *st, const uint32_t A[4],
                        const uint32_t B[4], uint64_t rho_q32, uint64_t guide_q32)
{
    int32_t K = pb->R * pb->D;
    orc_move mv;
    mv.reloc = ((uint64_t)A[0] < rho_q32);
    int guided = ((uint64_t)A[1] < guide_q32);
    if (!guided) {
        mv.i = pick(A[2], pb->N);
        mv.c1 = st->cell_of[mv.i];
        if (mv.reloc) { mv.i2 = -1; mv.c2 = pick(A[3], K); }
        else          { mv.i2 = pick(A[3], pb->N); mv.c2 = st->cell_of[mv.i2]; }
        return mv;
    }
    int32_t sa = pick(A[2], pb->N), sb = pick(A[3], pb->N);
    size_t rg = rowshard_of_cell(pb, st->cell_of[sa]);
    int64_t Ja = st->Afx[rg] + st->Efx[rg];
    int use_attention = ((u128)B[2] * (u128)(uint64_t)Ja) < ((u128)(uint64_t)st->Afx[rg] << 32);
    int64_t ka, kb;
    if (use_attention) {
        ka = cell_attention_key(pb, st, st->cell_of[sa]);
        kb = cell_attention_key(pb, st, st->cell_of[sb]);
    } else {
        ka = J_of_cell(pb, st, st->cell_of[sa]);
        kb = J_of_cell(pb, st, st->cell_of[sb]);
    }
    mv.i = (kb > ka) ? sb : sa;
    mv.c1 = st->cell_of[mv.i];
    if (mv.reloc) {
        int32_t ca = pick(B[0], K), cb = pick(B[1], K);
        int64_t ta = use_attention ? cell_attention_key(pb, st, ca) : J_of_cell(pb, st, ca);
        int64_t tb = use_attention ? cell_attention_key(pb, st, cb) : J_of_cell(pb, st, cb);
        mv.i2 = -1;
        mv.c2 = (tb < ta) ? cb : ca;
    } else {
        int32_t ta_s = pick(B[0], pb->N), tb_s = pick(B[1], pb->N);
        int64_t ta = use_attention ? cell_attention_key(pb, st, st->cell_of[ta_s])
                                   : J_of_cell(pb, st, st->cell_of[ta_s]);
        int64_t tb = use_attention ? cell_attention_key(pb, st, st->cell_of[tb_s])
                                   : J_of_cell(pb, st, st->cell_of[tb_s]);
        mv.i2 = (tb < ta) ? tb_s : ta_s;
        mv.c2 = st->cell_of[mv.i2];
    }
    return mv;
}

/* A proposal must stay inside the feasible set (Eqs. sample-bijection, nonempty-cell,
 * token-capacity): distinct cells, capacity kept in both cells, no cell emptied. */
static int feasible(const orc_problem *pb, const orc_state *st, const orc_move *mv)
{
    if (mv->c1 == mv->c2) return 0;
    int64_t ti = pb->t[mv->i];
    if (mv->reloc) {
        if (st->cnt[mv->c1] <= 1) return 0;
        return st->T[mv->c2] + ti <= pb->C;
    }
    int64_t t2 = pb->t[mv->i2];
    return st->T[mv->c1] - ti + t2 <= pb->C && st->T[mv->c2] - t2 + ti <= pb->C;
}

static void shift_sample(const orc_problem *pb, orc_state *st, int32_t i, int32_t from, int32_t to)
{
    int64_t ti = pb->t[i];
    size_t LP = (size_t)pb->L * pb->P;
    st->cell_of[i] = to;
    st->T[from] -= ti; st->Q[from] -= ti * ti; st->cnt[from] -= 1;
    st->T[to] += ti;   st->Q[to] += ti * ti;   st->cnt[to] += 1;
    size_t rg_from = rowshard_of_cell(pb, from), rg_to = rowshard_of_cell(pb, to);
    if (rg_from != rg_to) {
        int32_t *wf = st->W + rg_from * LP, *wt = st->W + rg_to * LP;
        const int32_t *qi = pb->q + (size_t)i * LP;
        for (size_t x = 0; x < LP; ++x) { wf[x] -= qi[x]; wt[x] += qi[x]; }
    }
}

/* IncrementalScore: move the sample(s), refresh the two cells' statistics and the
 * affected row-shards' rank loads, then rebuild the exact score from the cached terms. */
static void apply_move(const orc_problem *pb, orc_state *st, const orc_move *mv)
{
    shift_sample(pb, st, mv->i, mv->c1, mv->c2);
    if (!mv->reloc) shift_sample(pb, st, mv->i2, mv->c2, mv->c1);
    int32_t cells[2] = { mv->c1, mv->c2 };
    for (int x = 0; x < 2; ++x) {
        int32_t r = cells[x] / pb->D, g = pb->edp_of_dp[cells[x] % pb->D];
        st->Afx[(size_t)r * pb->G + g] = attention_fx(pb, st, r, g);
        st->Efx[(size_t)r * pb->G + g] = expert_fx(pb, st, r, g);
    }
    rescore_from_rows(pb, st);
}
/* Both move kinds are undone by sending every moved sample back where it came from. */
static void undo_move(const orc_problem *pb, orc_state *st, const orc_move *mv)
{
    orc_move back = *mv;
    back.c1 = mv->c2;
    back.c2 = mv->c1;
    apply_move(pb, st, &back);
}

/* Metropolis rule of Algorithm 3: accept when the score tuple improves, or when
 * u < exp(-max(Delta,0)/T) with Delta = (E' - E)/max(|E|,1).  In integers, with
 * u = (x+1)/2^32, tau = floor(T*ln2*2^32) and the paper's "1" equal to SC:
 *   Delta/T < -ln u   <=>   E' - E < ((tau * nl2(x)) >> 32) * max(E, SC) >> 32.
 * The accept word is drawn only when it is needed. */
int32_t orc_accept_uphill(int64_t e_old, int64_t e_new, int64_t SC, uint64_t tau, uint32_t x)
{
    int64_t dE = e_new - e_old;
    if (dE <= 0) return 1;
    u128 thr = ((u128)tau * orc_nl2(x)) >> 32;
    if (thr >> 62) return 1;                        /* absurdly hot: every move passes */
    int64_t M = e_old > SC ? e_old : SC;
    u128 bound = (thr * (u128)(uint64_t)M) >> 32;
    if (bound >> 63) return 1;                      /* saturated: certainly larger than dE */
    return (uint64_t)dE < (uint64_t)bound;
}

static int metropolis(const int64_t s_old[3], const int64_t s_new[3], int64_t SC, uint64_t tau,
                      uint64_t seed, uint32_t step, uint32_t level, uint32_t slot)
{
    if (lex_less(s_new, s_old)) return 1;
    int64_t e_old = energy(s_old), e_new = energy(s_new);
    if (e_new <= e_old) return 1;
    uint32_t X[4];
    draw(seed, step, level, slot, ORC_DRAW_ACCEPT, X);
    return orc_accept_uphill(e_old, e_new, SC, tau, X[0]);
}

/* Digest of a chain's accepted moves within a level (test instrumentation only). */
static inline uint64_t digest_step(uint64_t h, uint32_t step, const orc_move *mv)
{
    uint64_t second = mv->reloc ? (uint64_t)mv->c2 : (uint64_t)mv->i2;
    uint64_t code = ((uint64_t)mv->reloc << 63) ^ ((uint64_t)step << 40) ^ ((uint64_t)mv->i << 20) ^ second;
    return (h ^ code) * 0x100000001B3ull;
}

/* Per-level schedule integers derived from the geometric temperatures with IEEE double
 * operations only: tau_n = floor(T_n * ln2 * 2^32) and, for resampling,
 * cq_n = floor((1/T_{n+1} - 1/T_n) / ln2 * 2^16). */
void orc_schedule(int32_t n_levels, double t0, double t_ratio, uint64_t *tau, uint64_t *cq)
{
    const double LN2 = 0.6931471805599453094;
    double T = t0;
    for (int32_t n = 0; n < n_levels; ++n) {
        double Tnext = T * t_ratio;
        double x = T * LN2;
        x = x * 4294967296.0;
        tau[n] = (uint64_t)floor(x);
        double db = 1.0 / Tnext - 1.0 / T;
        double y = db * (1.0 / LN2);
        y = y * 65536.0;
        cq[n] = y > 0.0 ? (uint64_t)floor(y) : 0;
        T = Tnext;
    }
}

/* Systematic resampling with Boltzmann weights (Algorithm 3, resampling block):
 * normalised energy eq_j = (E_j - E_min) / max(E_min, SC) in Q32 (capped), exponent
 * z_j = eq_j * cq >> 16, weight w_j = 2^-z_j in Q32, cumulative F_j; with the offset
 * u0 = floor(x * F_total / 2^32) the m-th draw sits at u0 + m*F_total on a ruler of
 * length P*F_total and selects the first j whose P*F_j lies beyond it. */
void orc_resample(int32_t Ppop, const int64_t *E, int64_t SC, uint64_t cq, uint32_t x, int32_t *anc)
{
    int64_t Emin = E[0];
    for (int32_t j = 1; j < Ppop; ++j) if (E[j] < Emin) Emin = E[j];
    int64_t M = Emin > SC ? Emin : SC;
    uint64_t *F = (uint64_t *)malloc(sizeof(uint64_t) * Ppop);
    uint64_t run = 0;
    for (int32_t j = 0; j < Ppop; ++j) {
        u128 eq = ((u128)(uint64_t)(E[j] - Emin) << 32) / (u128)(uint64_t)M;
        if (eq > (((u128)1 << 48) - 1)) eq = ((u128)1 << 48) - 1;
        u128 z = (eq * (u128)cq) >> 16;
        if (z > ((u128)1 << 40)) z = (u128)1 << 40;
        run += orc_exp2neg((uint64_t)z);
        F[j] = run;
    }
    uint64_t Ftot = run;
    uint64_t u0 = (uint64_t)(((u128)x * Ftot) >> 32);
    int32_t j = 0;
    for (int32_t m = 0; m < Ppop; ++m) {
        u128 pos = (u128)u0 + (u128)m * Ftot;
        while ((u128)Ppop * F[j] <= pos) ++j;
        anc[m] = j;
    }
    free(F);
}

/* ------------------------------------------------------------------------------------ */
/* Fixed-row population annealing (Algorithm 3).                                         */
/*                                                                                        */
/* init_layouts [Ppop][N] is P_0.  Every level: each chain runs `steps` proposals at      */
/* temperature T_n from its slot's current state and reports its terminal state and its  */
/* trajectory-best state; the incumbent takes any strictly better trajectory-best        */
/* (chains scanned in slot order); unless it is the last level the population is         */
/* resampled from the terminal states.  Slot j always uses random stream j, whoever its  */
/* ancestor was.  full_rescore != 0 replaces the incremental update by a from-scratch    */
/* evaluation of the proposed layout (to show the two are the same thing).               */
/*                                                                                        */
/* Trace outputs (any may be NULL), per level n and slot j:                               */
/*   tr_term [n][j][3], tr_best [n][j][3] scores; tr_best_step [n][j] (0 = level start);  */
/*   tr_digest [n][j]; tr_anc [n][j] (levels 0..n_levels-2); tr_inc [n][3] incumbent.     */
/* counters[4] = proposed, feasible, accepted, improved-trajectory-best.                  */
/* Final outputs: best_layout [N], best_score [3], final_pop [Ppop][N] (last terminals).  */
/* ------------------------------------------------------------------------------------ */
int32_t orc_anneal(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C,
                   const int32_t *edp_of_dp, int32_t S, const double *alpha, const double *beta,
                   const int32_t *t, const int32_t *q,
                   int32_t Ppop, const int32_t *init_layouts,
                   int32_t n_levels, int32_t steps, double t0, double t_ratio,
                   double p_reloc, double p_guide, uint64_t seed,
                   int32_t full_rescore, int32_t n_threads,
                   int64_t *tr_term, int64_t *tr_best, int32_t *tr_best_step, uint64_t *tr_digest,
                   int32_t *tr_anc, int64_t *tr_inc, int64_t *counters,
                   int32_t *best_layout, int64_t *best_score, int32_t *final_pop)
{
    orc_problem pb;
    fill_problem(&pb, N, L, P, D, G, R, C, edp_of_dp, S, alpha, beta, t, q);
    const int64_t SC = ((int64_t)C * C) << ORC_FBITS;
    const uint64_t rho_q32 = (uint64_t)floor(p_reloc * 4294967296.0);
    const uint64_t guide_q32 = (uint64_t)floor(p_guide * 4294967296.0);
    uint64_t *tau = (uint64_t *)malloc(sizeof(uint64_t) * n_levels);
    uint64_t *cq = (uint64_t *)malloc(sizeof(uint64_t) * n_levels);
    orc_schedule(n_levels, t0, t_ratio, tau, cq);

    orc_state **pop = (orc_state **)malloc(sizeof(orc_state *) * Ppop);
    orc_state **nxt = (orc_state **)malloc(sizeof(orc_state *) * Ppop);
    orc_plan **best = (orc_plan **)malloc(sizeof(orc_plan *) * Ppop);
    for (int32_t j = 0; j < Ppop; ++j) {
        pop[j] = state_new(&pb); nxt[j] = state_new(&pb); best[j] = plan_new(&pb);
        memcpy(pop[j]->cell_of, init_layouts + (size_t)j * N, sizeof(int32_t) * N);
        evaluate(&pb, pop[j]);
    }
    /* incumbent = best seed (first of equals) */
    orc_plan *inc = plan_new(&pb);
    plan_take(&pb, inc, pop[0]->cell_of, pop[0]->s);
    for (int32_t j = 1; j < Ppop; ++j)
        if (lex_less(pop[j]->s, inc->s)) plan_take(&pb, inc, pop[j]->cell_of, pop[j]->s);
    int64_t seed_best[3] = { inc->s[0], inc->s[1], inc->s[2] };

    int64_t c_prop = 0, c_feas = 0, c_acc = 0, c_imp = 0;
    int64_t *Eterm = (int64_t *)malloc(sizeof(int64_t) * Ppop);
    int32_t *anc = (int32_t *)malloc(sizeof(int32_t) * Ppop);
    int32_t *bstep = (int32_t *)malloc(sizeof(int32_t) * Ppop);
    uint64_t *dig = (uint64_t *)malloc(sizeof(uint64_t) * Ppop);
    if (n_threads < 1) n_threads = 1;

    for (int32_t n = 0; n < n_levels; ++n) {
#pragma omp parallel for schedule(dynamic, 1) num_threads(n_threads) \
        reduction(+ : c_prop, c_feas, c_acc, c_imp)
        for (int32_t j = 0; j < Ppop; ++j) {
            orc_state *y = pop[j];
            orc_state *trial = full_rescore ? state_new(&pb) : NULL;
            plan_take(&pb, best[j], y->cell_of, y->s);
            bstep[j] = 0;
            uint64_t h = 0;
            for (int32_t k = 0; k < steps; ++k) {
                uint32_t A[4], B[4];
                draw(seed, (uint32_t)k, (uint32_t)n, (uint32_t)j, ORC_DRAW_A, A);
                draw(seed, (uint32_t)k, (uint32_t)n, (uint32_t)j, ORC_DRAW_B, B);
                orc_move mv = propose(&pb, y, A, B, rho_q32, guide_q32);
                ++c_prop;
                if (!feasible(&pb, y, &mv)) continue;
                ++c_feas;
                int64_t s_old[3] = { y->s[0], y->s[1], y->s[2] };
                int ok;
                if (full_rescore) {
                    memcpy(trial->cell_of, y->cell_of, sizeof(int32_t) * N);
                    trial->cell_of[mv.i] = mv.c2;
                    if (!mv.reloc) trial->cell_of[mv.i2] = mv.c1;
                    evaluate(&pb, trial);
                    ok = metropolis(s_old, trial->s, SC, tau[n], seed, (uint32_t)k, (uint32_t)n, (uint32_t)j);
                    if (ok) state_copy(&pb, y, trial);
                } else {
                    apply_move(&pb, y, &mv);
                    ok = metropolis(s_old, y->s, SC, tau[n], seed, (uint32_t)k, (uint32_t)n, (uint32_t)j);
                    if (!ok) undo_move(&pb, y, &mv);
                }
                if (!ok) continue;
                ++c_acc;
                h = digest_step(h, (uint32_t)k, &mv);
                if (lex_less(y->s, best[j]->s)) {
                    plan_take(&pb, best[j], y->cell_of, y->s);
                    bstep[j] = k + 1;
                    ++c_imp;
                }
            }
            dig[j] = h;
            if (trial) state_free(trial);
        }
        for (int32_t j = 0; j < Ppop; ++j) {
            size_t o = (size_t)n * Ppop + j;
            if (tr_term) memcpy(tr_term + o * 3, pop[j]->s, sizeof(int64_t) * 3);
            if (tr_best) memcpy(tr_best + o * 3, best[j]->s, sizeof(int64_t) * 3);
            if (tr_best_step) tr_best_step[o] = bstep[j];
            if (tr_digest) tr_digest[o] = dig[j];
            if (lex_less(best[j]->s, inc->s)) plan_take(&pb, inc, best[j]->cell_of, best[j]->s);
        }
        if (tr_inc) memcpy(tr_inc + (size_t)n * 3, inc->s, sizeof(int64_t) * 3);
        if (n < n_levels - 1) {
            uint32_t X[4];
            draw(seed, 0u, (uint32_t)n, 0u, ORC_DRAW_RESAMPLE, X);
            for (int32_t j = 0; j < Ppop; ++j) Eterm[j] = energy(pop[j]->s);
            orc_resample(Ppop, Eterm, SC, cq[n], X[0], anc);
            if (tr_anc) memcpy(tr_anc + (size_t)n * Ppop, anc, sizeof(int32_t) * Ppop);
            for (int32_t m = 0; m < Ppop; ++m) state_copy(&pb, nxt[m], pop[anc[m]]);
            orc_state **sw = pop; pop = nxt; nxt = sw;
        }
    }

    /* Validate(x*): coverage, capacity, nonempty cells, cached score == full rescoring,
     * and the non-regression assertion against the best seed. */
    int32_t status = 0;
    {
        orc_state *chk = state_new(&pb);
        memcpy(chk->cell_of, inc->cell_of, sizeof(int32_t) * N);
        for (int32_t i = 0; i < N; ++i) if (chk->cell_of[i] < 0 || chk->cell_of[i] >= R * D) status |= 1;
        if (!status) {
            evaluate(&pb, chk);
            for (int32_t c = 0; c < R * D; ++c) {
                if (chk->cnt[c] < 1) status |= 2;
                if (chk->T[c] > C) status |= 4;
            }
            if (memcmp(chk->s, inc->s, sizeof chk->s)) status |= 8;
            if (lex_less(seed_best, inc->s)) status |= 16;
        }
        state_free(chk);
    }
    if (best_layout) memcpy(best_layout, inc->cell_of, sizeof(int32_t) * N);
    if (best_score) memcpy(best_score, inc->s, sizeof(int64_t) * 3);
    if (final_pop)
        for (int32_t j = 0; j < Ppop; ++j) memcpy(final_pop + (size_t)j * N, pop[j]->cell_of, sizeof(int32_t) * N);
    if (counters) { counters[0] = c_prop; counters[1] = c_feas; counters[2] = c_acc; counters[3] = c_imp; }

    for (int32_t j = 0; j < Ppop; ++j) { state_free(pop[j]); state_free(nxt[j]); plan_free(best[j]); }
    plan_free(inc);
    free(pop); free(nxt); free(best); free(tau); free(cq); free(Eterm); free(anc); free(bstep); free(dig);
    return status;
}

/* ------------------------------------------------------------------------------------ */
/* Load-balance diagnostics of the evaluation section (Eq. global-ep-cv, the EP peak     */
/* sum and tail peak, Eq. ep-efficiency) for one layout.                                 */
/*   cv[0]: CV_global under the identity placement (expert e on rank e / H),            */
/*   cv[1]: CV_global under the given placement pi.                                      */
/*   peaks[0] = S_EP = sum_{r,l} max_{g,p} W,  peaks[1] = T_EP = max W,                  */
/*   peaks[2] = sum_{r,l} max_g sum_p W  (eta_EP = peaks[2] / (P * peaks[0])).           */
/*   att_joint[0] = sum_{r,g} A_{r,g}, att_joint[1] = max_g sum_r J_{r,g} (real units).  */
/* ------------------------------------------------------------------------------------ */
static double cv_of_loads(int32_t L, int32_t P, const int64_t *G)
{
    double acc = 0.0;
    for (int32_t l = 0; l < L; ++l) {
        double mean = 0.0;
        for (int32_t p = 0; p < P; ++p) mean += (double)G[(size_t)l * P + p];
        mean /= (double)P;
        double var = 0.0;
        for (int32_t p = 0; p < P; ++p) {
            double d = (double)G[(size_t)l * P + p] - mean;
            var += d * d;
        }
        var /= (double)P;
        acc += (mean > 0.0) ? sqrt(var) / mean : 0.0;
    }
    return acc / (double)L;
}

void orc_diagnostics(int32_t N, int32_t L, int32_t E, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C,
                     const int32_t *edp_of_dp, int32_t S, const double *alpha, const double *beta,
                     const int32_t *t, const int32_t *q, const int64_t *Lagg, const int32_t *pi,
                     const int32_t *cell_of, double cv[2], int64_t peaks[3], double att_joint[2], double *eta)
{
    int32_t H = E / P;
    int64_t *Gid = (int64_t *)calloc((size_t)L * P, sizeof(int64_t));
    int64_t *Gpi = (int64_t *)calloc((size_t)L * P, sizeof(int64_t));
    for (int32_t l = 0; l < L; ++l)
        for (int32_t e = 0; e < E; ++e) {
            Gid[(size_t)l * P + e / H] += Lagg[(size_t)l * E + e];
            Gpi[(size_t)l * P + pi[(size_t)l * E + e] / H] += Lagg[(size_t)l * E + e];
        }
    cv[0] = cv_of_loads(L, P, Gid);
    cv[1] = cv_of_loads(L, P, Gpi);
    free(Gid); free(Gpi);

    orc_problem pb;
    fill_problem(&pb, N, L, P, D, G, R, C, edp_of_dp, S, alpha, beta, t, q);
    orc_state *st = state_new(&pb);
    memcpy(st->cell_of, cell_of, sizeof(int32_t) * N);
    evaluate(&pb, st);
    int64_t s_ep = 0, t_ep = 0, n_ep = 0;
    for (int32_t r = 0; r < R; ++r)
        for (int32_t l = 0; l < L; ++l) {
            int64_t peak = 0, best_sum = 0;
            for (int32_t g = 0; g < G; ++g) {
                const int32_t *w = st->W + (((size_t)r * G + g) * L + l) * P;
                int64_t sum = 0;
                for (int32_t p = 0; p < P; ++p) { sum += w[p]; if (w[p] > peak) peak = w[p]; }
                if (sum > best_sum) best_sum = sum;
            }
            s_ep += peak;
            n_ep += best_sum;
            if (peak > t_ep) t_ep = peak;
        }
    peaks[0] = s_ep; peaks[1] = t_ep; peaks[2] = n_ep;
    *eta = s_ep > 0 ? (double)n_ep / ((double)P * (double)s_ep) : 1.0;
    const double SC = (double)(((int64_t)C * C) << ORC_FBITS);
    int64_t asum = 0;
    for (size_t x = 0; x < (size_t)R * G; ++x) asum += st->Afx[x];
    att_joint[0] = (double)asum / SC;
    att_joint[1] = (double)st->s[0] / SC;
    state_free(st);
}

/* ------------------------------------------------------------------------------------ */
/* Randomized fixed-row seeds (Algorithm 2, the trial loop without the pairing and       */
/* canonical-selection operators): one trial per population member.                      */
/*                                                                                        */
/* Reading of the two construction operators (the paper gives one sentence each):        */
/*  WindowShuffle: walk the samples in order (-t_i, i); keep a window of the next w       */
/*    not-yet-emitted samples; emit a uniformly chosen one of the window, close the gap   */
/*    (order kept) and refill from the sorted list.  Draw: Philox(h, 0, trial, 4).x for   */
/*    the h-th emitted sample, index = floor(x * window_size / 2^32).                     */
/*  RandomizedBestFit: the first K emitted samples open the K cells in order; each later  */
/*    sample looks at the cells it fits in, ranks them by (fuller first, then fewer       */
/*    samples, then lower index) and takes a uniformly chosen one of the leading          */
/*    min(w, #feasible).  Draw: Philox(h, 0, trial, 5).x.  No feasible cell: the trial    */
/*    is aborted.                                                                          */
/*  Cell b is (row b / D, slot b % D) (the pairing operator is not applied).              */
/* Member 0 is always the length-only seed; member j >= 1 is trial j, or the length-only  */
/* seed again when trial j aborted.  ok[j] = 1 when member j is its own trial's layout.   */
/* ------------------------------------------------------------------------------------ */
void orc_seed_trials(int32_t N, int32_t C, int32_t D, int32_t R, int32_t w, uint64_t seed, const int32_t *t,
                     const int32_t *seed_layout, int32_t Ppop, int32_t *layouts, int32_t *ok)
{
    int32_t K = R * D;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * N);
    for (int32_t i = 0; i < N; ++i) order[i] = i;
    for (int32_t x = 1; x < N; ++x) {               /* insertion sort by (-t, i) */
        int32_t s = order[x], y = x;
        while (y > 0 && (t[order[y - 1]] < t[s] || (t[order[y - 1]] == t[s] && order[y - 1] > s))) {
            order[y] = order[y - 1];
            --y;
        }
        order[y] = s;
    }
    int32_t *win = (int32_t *)malloc(sizeof(int32_t) * (w > 0 ? w : 1));
    int64_t *fill = (int64_t *)malloc(sizeof(int64_t) * K);
    int32_t *cnt = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * K);
    for (int32_t j = 0; j < Ppop; ++j) {
        int32_t *lay = layouts + (size_t)j * N;
        memcpy(lay, seed_layout, sizeof(int32_t) * N);
        ok[j] = (j == 0);
        if (j == 0) continue;
        int32_t nwin = 0, next = 0, good = 1;
        for (int32_t b = 0; b < K; ++b) { fill[b] = 0; cnt[b] = 0; }
        for (int32_t h = 0; h < N && good; ++h) {
            while (nwin < w && next < N) win[nwin++] = order[next++];
            uint32_t X[4];
            draw(seed, (uint32_t)h, 0u, (uint32_t)j, 4u, X);
            int32_t pos = pick(X[0], nwin);
            int32_t s = win[pos];
            for (int32_t x = pos; x + 1 < nwin; ++x) win[x] = win[x + 1];
            --nwin;
            int32_t b;
            if (h < K) b = h;
            else {
                int32_t nc = 0;
                for (int32_t c = 0; c < K; ++c) if (fill[c] + t[s] <= C) cand[nc++] = c;
                if (nc == 0) { good = 0; break; }
                /* order the feasible cells: fuller first, then fewer samples, then lower index */
                for (int32_t x = 1; x < nc; ++x) {
                    int32_t c = cand[x], y = x;
                    while (y > 0) {
                        int32_t p = cand[y - 1];
                        int before = (fill[p] > fill[c]) || (fill[p] == fill[c] && (cnt[p] < cnt[c] || (cnt[p] == cnt[c] && p < c)));
                        if (before) break;
                        cand[y] = p;
                        --y;
                    }
                    cand[y] = c;
                }
                draw(seed, (uint32_t)h, 0u, (uint32_t)j, 5u, X);
                b = cand[pick(X[0], nc < w ? nc : w)];
            }
            fill[b] += t[s];
            cnt[b] += 1;
            lay[s] = b;
        }
        if (good) ok[j] = 1;
        else memcpy(lay, seed_layout, sizeof(int32_t) * N);
    }
    free(order); free(win); free(fill); free(cnt); free(cand);
}

/* ------------------------------------------------------------------------------------ */
/* EDPAwarePair (Section 4.1.1, the third construction operator of Algorithm 2): keeps   */
/* every completed cell as a set of samples and only changes which (row, DP slot) it     */
/* occupies.                                                                              */
/*                                                                                        */
/* Reading (the paper gives one sentence; "parity unpinned" against the paper for the     */
/* sampling law, the rest is pinned by a worked example and closed forms):                */
/*  * profile of a cell b: w_b[l][p] = sum of q[i][l][p] over its samples; its            */
/*    routed-token peak is max_{l,p} w_b[l][p].  Cells are taken in order of decreasing   */
/*    peak, ties by lower cell index.                                                     */
/*  * V[r][g][l][p] is the rank load of row-shard (r, g) from the cells placed so far.    */
/*    For the cell in hand every still-empty slot s = r*D + d (shard g = edp(d)) gets the */
/*    insertion key (sum_l max_p (V+w) - sum_l max_p V,  max_{l,p} (V+w)); slots are      */
/*    ranked by ascending key, ties by lower slot index.                                  */
/*  * rank-decaying top-w sampling: with m = min(w, #empty), rank rho = min(m-1, number   */
/*    of leading zero bits of the draw) - rank 0 with probability 1/2, rank 1 with 1/4,   */
/*    ..., the remainder on rank m-1.  Draw: Philox(h, 0, trial, 6).x for the h-th cell   */
/*    placed.                                                                             */
/* Member 0 is left untouched (the length-only seed); member j >= 1 is trial j.           */
/* ------------------------------------------------------------------------------------ */
void orc_edp_pair(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t w, uint64_t seed,
                  const int32_t *q, const int32_t *edp_of_dp, int32_t Ppop, int32_t *layouts)
{
    const int32_t K = R * D;
    const size_t LP = (size_t)L * P;
    int64_t *prof = (int64_t *)malloc(sizeof(int64_t) * K * LP);
    int64_t *V = (int64_t *)malloc(sizeof(int64_t) * (size_t)R * G * LP);
    int64_t *peak = (int64_t *)malloc(sizeof(int64_t) * K);
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *slot_of = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *empty = (int32_t *)malloc(sizeof(int32_t) * K);
    int32_t *rank = (int32_t *)malloc(sizeof(int32_t) * K);
    int64_t *kd = (int64_t *)malloc(sizeof(int64_t) * K), *kp = (int64_t *)malloc(sizeof(int64_t) * K);
    for (int32_t j = 1; j < Ppop; ++j) {
        int32_t *lay = layouts + (size_t)j * N;
        memset(prof, 0, sizeof(int64_t) * K * LP);
        memset(V, 0, sizeof(int64_t) * (size_t)R * G * LP);
        for (int32_t i = 0; i < N; ++i)
            for (size_t x = 0; x < LP; ++x) prof[(size_t)lay[i] * LP + x] += q[(size_t)i * LP + x];
        for (int32_t b = 0; b < K; ++b) {
            int64_t m = 0;
            for (size_t x = 0; x < LP; ++x) if (prof[(size_t)b * LP + x] > m) m = prof[(size_t)b * LP + x];
            peak[b] = m;
            order[b] = b;
            empty[b] = 1;
        }
        for (int32_t x = 1; x < K; ++x) {                /* insertion sort by (-peak, b) */
            int32_t s = order[x], y = x;
            while (y > 0 && (peak[order[y - 1]] < peak[s] || (peak[order[y - 1]] == peak[s] && order[y - 1] > s))) {
                order[y] = order[y - 1];
                --y;
            }
            order[y] = s;
        }
        for (int32_t h = 0; h < K; ++h) {
            const int32_t b = order[h];
            const int64_t *wb = prof + (size_t)b * LP;
            int32_t ne = 0;
            for (int32_t s = 0; s < K; ++s) {
                if (!empty[s]) continue;
                const int32_t r = s / D, g = edp_of_dp[s % D];
                const int64_t *v = V + ((size_t)r * G + g) * LP;
                int64_t e_old = 0, e_new = 0, pk = 0;
                for (int32_t l = 0; l < L; ++l) {
                    int64_t mo = 0, mn = 0;
                    for (int32_t p = 0; p < P; ++p) {
                        const int64_t a = v[(size_t)l * P + p], c = a + wb[(size_t)l * P + p];
                        if (a > mo) mo = a;
                        if (c > mn) mn = c;
                    }
                    e_old += mo;
                    e_new += mn;
                    if (mn > pk) pk = mn;
                }
                kd[s] = e_new - e_old;
                kp[s] = pk;
                /* insert s into the ranking: ascending (kd, kp, s) */
                int32_t y = ne++;
                while (y > 0) {
                    const int32_t o = rank[y - 1];
                    if (kd[o] < kd[s] || (kd[o] == kd[s] && (kp[o] < kp[s] || (kp[o] == kp[s] && o < s)))) break;
                    rank[y] = o;
                    --y;
                }
                rank[y] = s;
            }
            uint32_t X[4];
            draw(seed, (uint32_t)h, 0u, (uint32_t)j, 6u, X);
            int32_t lz = 0;
            while (lz < 32 && !((X[0] >> (31 - lz)) & 1u)) ++lz;
            const int32_t m = ne < w ? ne : w;
            const int32_t rho = lz < m - 1 ? lz : m - 1;
            const int32_t s = rank[rho];
            slot_of[b] = s;
            empty[s] = 0;
            int64_t *v = V + ((size_t)(s / D) * G + edp_of_dp[s % D]) * LP;
            for (size_t x = 0; x < LP; ++x) v[x] += wb[x];
        }
        for (int32_t i = 0; i < N; ++i) lay[i] = slot_of[lay[i]];
    }
    free(prof); free(V); free(peak); free(order); free(slot_of); free(empty); free(rank); free(kd); free(kp);
}

/* ------------------------------------------------------------------------------------ */
/* Canonicalize / CanonicalMap / QualityDiversitySelect (Section 4.1.1, Algorithm 2).    */
/*                                                                                        */
/* Canonicalize: layouts that differ only by the order of rows, or by which of the       */
/* exchangeable DP slots of one EDP shard a cell sits in, get the same signature.  A cell */
/* is named by its smallest sample id (sample order inside a cell is not represented at   */
/* all); inside a row the cells of one shard are listed by that name over the shard's     */
/* slots in increasing slot order; rows are listed by their smallest sample id.  Any      */
/* other total order would give the same classes.                                         */
/* ------------------------------------------------------------------------------------ */
void orc_canonicalize(int32_t N, int32_t D, int32_t G, int32_t R, const int32_t *edp_of_dp,
                      const int32_t *lay, int32_t *canon)
{
    const int32_t K = R * D;
    int32_t *name = (int32_t *)malloc(sizeof(int32_t) * K);       /* smallest sample of the cell */
    int32_t *new_d = (int32_t *)malloc(sizeof(int32_t) * K);      /* slot inside the row */
    int32_t *rname = (int32_t *)malloc(sizeof(int32_t) * R);
    int32_t *new_r = (int32_t *)malloc(sizeof(int32_t) * R);
    for (int32_t c = 0; c < K; ++c) name[c] = N;
    for (int32_t i = N - 1; i >= 0; --i) name[lay[i]] = i;
    for (int32_t r = 0; r < R; ++r) {
        rname[r] = N;
        for (int32_t d = 0; d < D; ++d) if (name[r * D + d] < rname[r]) rname[r] = name[r * D + d];
        for (int32_t g = 0; g < G; ++g)
            for (int32_t d = 0; d < D; ++d) {
                if (edp_of_dp[d] != g) continue;
                /* position of cell (r, d) among the cells of shard g in this row, by name */
                int32_t pos = 0;
                for (int32_t d2 = 0; d2 < D; ++d2)
                    if (edp_of_dp[d2] == g && name[r * D + d2] < name[r * D + d]) ++pos;
                /* the pos-th slot of the shard */
                int32_t seen = 0, target = -1;
                for (int32_t d2 = 0; d2 < D && target < 0; ++d2)
                    if (edp_of_dp[d2] == g) { if (seen == pos) target = d2; ++seen; }
                new_d[r * D + d] = target;
            }
    }
    for (int32_t r = 0; r < R; ++r) {
        int32_t pos = 0;
        for (int32_t r2 = 0; r2 < R; ++r2) if (rname[r2] < rname[r]) ++pos;
        new_r[r] = pos;
    }
    for (int32_t i = 0; i < N; ++i) canon[i] = new_r[lay[i] / D] * D + new_d[lay[i]];
    free(name); free(new_d); free(rname); free(new_r);
}

/* Co-assignment distance of two labelings in Q20: 1 - |pairs together in both| / |pairs
 * together in either| (0 when neither puts any two samples together). */
int64_t orc_coassign_q20(int32_t N, const int32_t *la, const int32_t *lb)
{
    int64_t pa = 0, pb = 0, both = 0;
    for (int32_t i = 0; i < N; ++i)
        for (int32_t i2 = i + 1; i2 < N; ++i2) {
            const int sa = la[i] == la[i2], sb = lb[i] == lb[i2];
            pa += sa; pb += sb; both += (sa && sb);
        }
    const int64_t uni = pa + pb - both;
    if (uni == 0) return 0;
    return ((int64_t)1 << 20) - (both << 20) / uni;
}

/* Sorted projections of the row features (the Sliced-Wasserstein sketch), phi [nproj][R].
 * Row features in Q16 (F = 2 + G*L of them):
 *   tokens / (C*D),  sum of squared lengths / (C*C*D),  and for every shard g and layer l the
 *   busiest rank of row-shard (r, g), max_p W[r][g][l][p] / (k * C * |D_g|).
 * Projection k has entries +1 / -1: -1 where the top bit of Philox(f, 0, k, 7).x is set. */
void orc_sw_sketch(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C, int32_t k,
                   int32_t nproj, uint64_t seed, const int32_t *t, const int32_t *q, const int32_t *edp_of_dp,
                   const int32_t *lay, int64_t *phi)
{
    const int32_t F = 2 + G * L;
    const size_t LP = (size_t)L * P;
    int64_t *H = (int64_t *)calloc((size_t)R * F, sizeof(int64_t));
    int64_t *W = (int64_t *)calloc((size_t)R * G * LP, sizeof(int64_t));
    int64_t *Tr = (int64_t *)calloc(R, sizeof(int64_t)), *Qr = (int64_t *)calloc(R, sizeof(int64_t));
    int32_t *ng = (int32_t *)calloc(G, sizeof(int32_t));
    for (int32_t d = 0; d < D; ++d) ng[edp_of_dp[d]] += 1;
    for (int32_t i = 0; i < N; ++i) {
        const int32_t r = lay[i] / D, g = edp_of_dp[lay[i] % D];
        Tr[r] += t[i];
        Qr[r] += (int64_t)t[i] * t[i];
        for (size_t x = 0; x < LP; ++x) W[((size_t)r * G + g) * LP + x] += q[(size_t)i * LP + x];
    }
    for (int32_t r = 0; r < R; ++r) {
        H[(size_t)r * F + 0] = (int64_t)(((unsigned __int128)Tr[r] << 16) / ((unsigned __int128)C * D));
        H[(size_t)r * F + 1] = (int64_t)(((unsigned __int128)Qr[r] << 16) / ((unsigned __int128)C * C * D));
        for (int32_t g = 0; g < G; ++g)
            for (int32_t l = 0; l < L; ++l) {
                int64_t m = 0;
                for (int32_t p = 0; p < P; ++p) {
                    const int64_t v = W[((size_t)r * G + g) * LP + (size_t)l * P + p];
                    if (v > m) m = v;
                }
                H[(size_t)r * F + 2 + g * L + l] = (m << 16) / ((int64_t)k * C * ng[g]);
            }
    }
    for (int32_t kk = 0; kk < nproj; ++kk) {
        int64_t *ph = phi + (size_t)kk * R;
        for (int32_t r = 0; r < R; ++r) ph[r] = 0;
        for (int32_t f = 0; f < F; ++f) {
            uint32_t X[4];
            draw(seed, (uint32_t)f, 0u, (uint32_t)kk, 7u, X);
            const int64_t sgn = (X[0] >> 31) ? -1 : 1;
            for (int32_t r = 0; r < R; ++r) ph[r] += sgn * H[(size_t)r * F + f];
        }
        for (int32_t x = 1; x < R; ++x) {              /* insertion sort, ascending */
            int64_t v = ph[x];
            int32_t y = x;
            while (y > 0 && ph[y - 1] > v) { ph[y] = ph[y - 1]; --y; }
            ph[y] = v;
        }
    }
    free(H); free(W); free(Tr); free(Qr); free(ng);
}

/* Plan distance in Q20 units (0 .. about 3 * 2^20): cell co-assignment + row co-assignment +
 * sketch distance floor(16 * sum_k sum_r |phi_k(x)[r] - phi_k(y)[r]| / (nproj * R * F)).
 * The paper names the three ingredients but not how they are mixed: equal weights here. */
int64_t orc_plan_distance(int32_t N, int32_t D, int32_t R, int32_t F, int32_t nproj, const int32_t *la,
                          const int32_t *lb, const int64_t *phia, const int64_t *phib)
{
    int32_t *ra = (int32_t *)malloc(sizeof(int32_t) * N), *rb = (int32_t *)malloc(sizeof(int32_t) * N);
    for (int32_t i = 0; i < N; ++i) { ra[i] = la[i] / D; rb[i] = lb[i] / D; }
    int64_t d = orc_coassign_q20(N, la, lb) + orc_coassign_q20(N, ra, rb);
    int64_t s = 0;
    for (size_t x = 0; x < (size_t)nproj * R; ++x) s += phia[x] > phib[x] ? phia[x] - phib[x] : phib[x] - phia[x];
    d += (s * 16) / ((int64_t)nproj * R * F);
    free(ra); free(rb);
    return d;
}

/* CanonicalMap + QualityDiversitySelect over the population as the candidate set.
 *  - members with the same signature form one class; its representative has the lowest score
 *    (lexicographic), ties by lower member index;
 *  - the selection starts from the representative with the lowest score and then repeatedly
 *    takes the representative x that maximises  min_{y selected} d(x, y) - (eta * delta0(x)),
 *    delta0(x) = floor((S0(x) - S0*) * 2^20 / S0*) the primary-score gap to the winner in Q20,
 *    eta given in Q16, ties by lower member index;
 *  - new member m is the (m mod n_distinct)-th selected representative.
 * order [Ppop]: selected member indices (first *n_distinct valid); layouts are rewritten.
 * dist (nullable) [Ppop][Ppop]: plan distances between members (all pairs). */
void orc_select_population(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C, int32_t k,
                           int32_t nproj, int64_t eta_q16, uint64_t seed, const int32_t *t, const int32_t *q,
                           const int32_t *edp_of_dp, int32_t Ppop, const int64_t *scores, int32_t *layouts,
                           int32_t *n_distinct, int32_t *order, int64_t *dist)
{
    const int32_t F = 2 + G * L;
    int32_t *canon = (int32_t *)malloc(sizeof(int32_t) * (size_t)Ppop * N);
    int64_t *phi = (int64_t *)malloc(sizeof(int64_t) * (size_t)Ppop * nproj * R);
    int32_t *rep = (int32_t *)malloc(sizeof(int32_t) * Ppop), *sel = (int32_t *)calloc(Ppop, sizeof(int32_t));
    int64_t *mind = (int64_t *)malloc(sizeof(int64_t) * Ppop), *pen = (int64_t *)malloc(sizeof(int64_t) * Ppop);
    for (int32_t j = 0; j < Ppop; ++j) {
        orc_canonicalize(N, D, G, R, edp_of_dp, layouts + (size_t)j * N, canon + (size_t)j * N);
        orc_sw_sketch(N, L, P, D, G, R, C, k, nproj, seed, t, q, edp_of_dp, layouts + (size_t)j * N,
                      phi + (size_t)j * nproj * R);
    }
#define LEXLT(a, b) ((a)[0] != (b)[0] ? (a)[0] < (b)[0] : ((a)[1] != (b)[1] ? (a)[1] < (b)[1] : (a)[2] < (b)[2]))
    for (int32_t j = 0; j < Ppop; ++j) {
        rep[j] = 1;
        for (int32_t o = 0; o < Ppop && rep[j]; ++o) {
            if (o == j || memcmp(canon + (size_t)j * N, canon + (size_t)o * N, sizeof(int32_t) * N) != 0) continue;
            const int64_t *sj = scores + 3 * (size_t)j, *so = scores + 3 * (size_t)o;
            if (LEXLT(so, sj) || (!LEXLT(sj, so) && o < j)) rep[j] = 0;
        }
    }
    if (dist)
        for (int32_t a = 0; a < Ppop; ++a)
            for (int32_t b = 0; b < Ppop; ++b)
                dist[(size_t)a * Ppop + b] = orc_plan_distance(N, D, R, F, nproj, layouts + (size_t)a * N, layouts + (size_t)b * N,
                                                               phi + (size_t)a * nproj * R, phi + (size_t)b * nproj * R);
    int32_t nd = 0, best = -1;
    for (int32_t j = 0; j < Ppop; ++j) {
        if (!rep[j]) continue;
        ++nd;
        if (best < 0 || LEXLT(scores + 3 * (size_t)j, scores + 3 * (size_t)best)) best = j;
    }
    const int64_t s0 = scores[3 * (size_t)best];
    for (int32_t j = 0; j < Ppop; ++j)
        pen[j] = s0 > 0 ? (int64_t)(((unsigned __int128)(((unsigned __int128)(uint64_t)(scores[3 * (size_t)j] - s0) << 20) / (uint64_t)s0)
                                     * (unsigned __int128)(uint64_t)eta_q16) >> 16) : 0;
    int32_t last = best;
    for (int32_t n = 0; n < nd; ++n) {
        order[n] = last;
        sel[last] = 1;
        int32_t nxt = -1;
        int64_t bestv = 0;
        for (int32_t j = 0; j < Ppop; ++j) {
            if (!rep[j] || sel[j]) continue;
            const int64_t dj = orc_plan_distance(N, D, R, F, nproj, layouts + (size_t)j * N, layouts + (size_t)last * N,
                                                 phi + (size_t)j * nproj * R, phi + (size_t)last * nproj * R);
            if (n == 0 || dj < mind[j]) mind[j] = dj;
            const int64_t v = mind[j] - pen[j];
            if (nxt < 0 || v > bestv) { nxt = j; bestv = v; }
        }
        last = nxt;
    }
#undef LEXLT
    int32_t *old = (int32_t *)malloc(sizeof(int32_t) * (size_t)Ppop * N);
    memcpy(old, layouts, sizeof(int32_t) * (size_t)Ppop * N);
    for (int32_t m = 0; m < Ppop; ++m) memcpy(layouts + (size_t)m * N, old + (size_t)order[m % nd] * N, sizeof(int32_t) * N);
    for (int32_t m = nd; m < Ppop; ++m) order[m] = order[m % nd];
    *n_distinct = nd;
    free(old); free(canon); free(phi); free(rep); free(sel); free(mind); free(pen);
}

/* ------------------------------------------------------------------------------------ */
/* Thin windows onto two internal functions, so that tests can pin them one call at a    */
/* time (they add no arithmetic: the chain loop above calls the same propose() and       */
/* energy()).                                                                            */
/*   orc_propose_once: GuidedProposal (Section 4.1.2) on the state of `cell_of` with the */
/*   given random words; move = {reloc, i, i2, c1, c2}; returns feasibility (0/1).       */
/*   orc_energy: Eq. pa-energy of a score tuple.                                         */
/* ------------------------------------------------------------------------------------ */
int32_t orc_propose_once(int32_t N, int32_t L, int32_t P, int32_t D, int32_t G, int32_t R, int32_t C,
                         const int32_t *edp_of_dp, int32_t S, const double *alpha, const double *beta,
                         const int32_t *t, const int32_t *q, const int32_t *cell_of,
                         const uint32_t A[4], const uint32_t B[4], uint64_t rho_q32, uint64_t guide_q32,
                         int32_t move[5])
{
    orc_problem pb;
    fill_problem(&pb, N, L, P, D, G, R, C, edp_of_dp, S, alpha, beta, t, q);
    orc_state *st = state_new(&pb);
    memcpy(st->cell_of, cell_of, sizeof(int32_t) * N);
    evaluate(&pb, st);
    orc_move mv = propose(&pb, st, A, B, rho_q32, guide_q32);
    int32_t ok = feasible(&pb, st, &mv);
    move[0] = mv.reloc; move[1] = mv.i; move[2] = mv.i2; move[3] = mv.c1; move[4] = mv.c2;
    state_free(st);
    return ok;
}

int64_t orc_energy(const int64_t s[3]) { return energy(s); }
