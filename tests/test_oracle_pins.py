"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test names the passage (section, equation, algorithm or figure) it leans on.
"""
import itertools
import math
import os
from decimal import Decimal, getcontext, ROUND_FLOOR

import numpy as np
import pytest

import oracle
from paper_2608_12146_b200.windows import custom_spec, make_window

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------------------
# helpers written differently from the oracle (matrix form, Python integers)
# ----------------------------------------------------------------------------------------
def score_matrix_form(t, q, cell_of, R, D, edp, C, alpha=(1.0, 1.0), beta=(0.0, 1.0)):
    """Score tuple (Eq. lexicographic-score) in exact Python integers scaled by 2^8*C^2."""
    t = np.asarray(t, dtype=object)
    N = len(t)
    G = max(edp) + 1
    K = R * D
    X = np.zeros((N, K), dtype=object)
    X[np.arange(N), cell_of] = 1
    T = X.T @ t
    Q = X.T @ (t * t)
    ah = [int(math.floor(a * 256 + 0.5)) for a in alpha]
    bh = [int(math.floor(b * 256 + 0.5)) for b in beta]
    J = {}
    for r in range(R):
        for g in range(G):
            cells = [r * D + d for d in range(D) if edp[d] == g]
            A = sum(max(ah[s] * C * T[c] + bh[s] * Q[c] for c in cells) for s in range(len(ah)))
            members = [i for i in range(N) if cell_of[i] in cells]
            W = np.asarray(q, dtype=object)[members].sum(axis=0) if members else 0 * np.asarray(q[0], dtype=object)
            E = 256 * C * sum(int(max(row)) for row in W)
            J[(r, g)] = int(A) + int(E)
    U = [sum(J[(r, g)] for r in range(R)) for g in range(G)]
    return (max(U), sum(U), max(J.values()))


def hetero_window(N=48, L=3, E=8, k=2, C=2048, D=4, P=4, seed=7):
    return make_window(custom_spec("pin", N, L, E, k, C, D, P, 4, 100, data_seed=seed))


def placed(w):
    s = w.spec
    pi, G = oracle.lpt(oracle.aggregate(w.demand), s.ep_width)
    return pi, G, oracle.project(w.demand, pi, s.ep_width)


# ----------------------------------------------------------------------------------------
# random numbers and integer transcendental functions
# ----------------------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt")) if l[0] not in "#\n"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert oracle.philox4x32_10(v[0:4], v[4:6]).tolist() == v[6:10]


def test_philox_counter_and_key_sensitivity():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] += 1
        assert (oracle.philox4x32_10(c, [5, 6]) != base).all()
    assert (oracle.philox4x32_10([1, 2, 3, 4], [5, 7]) != base).all()


def test_nl2_matches_log2():
    rng = np.random.default_rng(0)
    xs = list(rng.integers(0, 2 ** 32, 3000)) + [0, 1, 2, 3, 2 ** 31 - 1, 2 ** 31, 2 ** 32 - 2, 2 ** 32 - 1]
    for x in xs:
        want = 32.0 - math.log2(int(x) + 1)
        got = oracle.nl2(int(x)) / 2.0 ** 32
        # 24 fraction bits, truncated: the oracle may sit above the truth by < 2^-24
        assert -1e-12 <= got - want < 2.0 ** -24 + 1e-12
    for e in range(33):      # exact at powers of two
        assert oracle.nl2(2 ** e - 1) == (32 - e) << 32
    assert oracle.nl2(2 ** 32 - 1) == 0


def test_exp2_table_against_high_precision():
    getcontext().prec = 80
    for i, have in enumerate(oracle.exp2_table(), start=1):
        v = (Decimal(2) ** (-(Decimal(1) / Decimal(2 ** i)))) * Decimal(2 ** 63)
        assert int(have) == int(v.to_integral_value(rounding=ROUND_FLOOR))


def test_exp2neg_matches_pow():
    rng = np.random.default_rng(1)
    assert oracle.exp2neg(0) == 2 ** 32
    assert oracle.exp2neg(32 << 32) == 0 and oracle.exp2neg(2 ** 40) == 0
    for n in range(32):
        assert oracle.exp2neg(n << 32) == 2 ** (32 - n)
    for z in rng.integers(0, 20 << 32, 3000):
        want = 2.0 ** (-int(z) / 2.0 ** 32)
        got = oracle.exp2neg(int(z)) / 2.0 ** 32
        # truncated products and 2^-24 exponent quantisation: relative error below 2^-22, never
        # more than one output unit below the truth
        assert got >= want - 2.0 ** -32 - want * 2.0 ** -40
        assert got <= want * (1 + 2.0 ** -22) + 2.0 ** -32


def test_schedule_integers():
    tau, cq = oracle.schedule(5, 1e-3, 0.5)
    T = 1e-3
    for n in range(5):
        assert abs(int(tau[n]) - T * math.log(2) * 2 ** 32) <= 1
        want_cq = (1.0 / (T * 0.5) - 1.0 / T) / math.log(2) * 65536
        assert abs(int(cq[n]) - want_cq) <= 1e-6 * want_cq + 1
        T *= 0.5


def test_metropolis_frequency_follows_exp():
    """Algorithm 3: an uphill move passes with probability exp(-Delta/T)."""
    rng = np.random.default_rng(2)
    SC = oracle.score_scale(4096)
    T = 2e-3
    tau = int(oracle.schedule(1, T, 1.0)[0][0])
    e_old = 70 * SC
    n = 40000
    xs = rng.integers(0, 2 ** 32, n)
    for ratio in (0.1, 0.7, 2.0, 5.0):                 # Delta / T
        dE = int(ratio * T * e_old)
        hits = sum(oracle.accept_uphill(e_old, e_old + dE, SC, tau, int(x)) for x in xs)
        p = math.exp(-ratio)
        assert abs(hits / n - p) < 4 * math.sqrt(p * (1 - p) / n) + 1e-4
    # the paper's max(|E|,1): below SC the normaliser is SC itself
    small = SC // 10
    dE = int(0.7 * T * SC)
    hits = sum(oracle.accept_uphill(small, small + dE, SC, tau, int(x)) for x in xs)
    assert abs(hits / n - math.exp(-0.7)) < 0.011
    # downhill or level always passes; zero temperature never passes uphill
    assert oracle.accept_uphill(e_old, e_old, SC, tau, 123)
    assert not any(oracle.accept_uphill(e_old, e_old + 1, SC, 0, int(x)) for x in xs[:500])


# ----------------------------------------------------------------------------------------
# aggregate demand, Algorithm 1, projection
# ----------------------------------------------------------------------------------------
def read_fig2():
    a, meta = [], {}
    for line in open(os.path.join(GOLD, "fig2_instance.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, val = line.split(":")
        nums = [int(x) for x in val.split()]
        if key.startswith("sample"):
            a.append(nums)
        else:
            meta[key.strip()] = nums
    return np.array(a, dtype=np.int32)[:, None, :], meta


def test_fig2_placement_and_row_peaks():
    a, m = read_fig2()                     # [4][1][4]
    Lagg = oracle.aggregate(a)
    assert Lagg.tolist() == [[6, 6, 2, 2]]
    ident = np.arange(4, dtype=np.int32)[None, :]
    assert oracle.project(a, ident, 2).sum(axis=0).tolist() == [m["window_load_identity"]]
    pi, G = oracle.lpt(Lagg, 2)
    assert pi.tolist() == [[0, 2, 1, 3]] and G.tolist() == [m["window_load_lpt"]]
    t = np.full(4, 4, np.int32)
    for placement, packing, key in ((ident, "packing_A_rows", "row_peak_identity"),
                                    (ident, "packing_B_rows", "row_peak_identity"),
                                    (pi, "packing_A_rows", "row_peaks_lpt_packing_A"),
                                    (pi, "packing_B_rows", "row_peaks_lpt_packing_B")):
        q = oracle.project(a, placement, 2)
        ev = oracle.eval_layouts(t, q, np.array(m[packing], np.int32), R=2, C_cap=8, D=1)
        assert ev["W"][0].max(axis=(1, 2, 3)).tolist() == m[key]


def test_fig2_objective_by_hand():
    """alpha=(1,1), beta=(0,1), C=8: each row has Tbar=1, Qbar=2*(1/2)^2=1/2, so A=1+1.5=2.5;
    E = row peak / C = 1 (packing A) or 1/2 (packing B); G=1 so U = J_0 + J_1."""
    a, m = read_fig2()
    pi, _ = oracle.lpt(oracle.aggregate(a), 2)
    q = oracle.project(a, pi, 2)
    t = np.full(4, 4, np.int32)
    SC = oracle.score_scale(8)
    for packing, want in (("packing_A_rows", (7.0, 7.0, 3.5)), ("packing_B_rows", (6.0, 6.0, 3.0))):
        lay = np.array(m[packing], np.int32)
        ev = oracle.eval_layouts(t, q, lay, R=2, C_cap=8, D=1)
        assert (ev["score"][0] / SC).tolist() == list(want)
        assert oracle.eval_f64(t, q, lay, R=2, C_cap=8, D=1).tolist() == list(want)


def test_objective_by_hand_two_slots():
    """One row, two DP slots, C=10, t=(6,2,3,5); cells {0,1} and {2,3}.
    One shard: stage maxima 0.8 and max(0.8+0.40, 0.8+0.34)=1.2, A=2.0; W=(12,4), E=1.2; J=3.2.
    Two shards: J_0 = 0.8+1.2+0.6 = 2.6, J_1 = 0.8+1.14+0.6 = 2.54."""
    t = np.array([6, 2, 3, 5], np.int32)
    q = np.array([[[6, 0]], [[0, 2]], [[1, 2]], [[5, 0]]], np.int32)
    lay = np.array([0, 0, 1, 1], np.int32)
    SC = oracle.score_scale(10)
    one = oracle.eval_layouts(t, q, lay, R=1, C_cap=10, D=2, edp_of_dp=[0, 0])
    assert one["score"][0].tolist() == [int(3.2 * SC + 0.5)] * 3
    two = oracle.eval_layouts(t, q, lay, R=1, C_cap=10, D=2, edp_of_dp=[0, 1])
    assert two["score"][0].tolist() == [round(2.6 * SC), round(5.14 * SC), round(2.6 * SC)]
    np.testing.assert_allclose(oracle.eval_f64(t, q, lay, 1, 10, 2, [0, 1]), [2.6, 5.14, 2.6], rtol=1e-14)


def test_lpt_tie_breaks_and_equal_loads():
    """Algorithm 1: argsort by (-L, e), argmin by (G, p), exactly H experts per rank.
    With all loads equal the visit order is e = 0,1,2,... and ranks fill round-robin,
    so pi(e) = (e mod P)*H + e div P."""
    for E, P in ((8, 4), (16, 4), (12, 3), (6, 6), (5, 1)):
        H = E // P
        pi, G = oracle.lpt(np.full((1, E), 7, np.int64), P)
        assert pi[0].tolist() == [(e % P) * H + e // P for e in range(E)]
        assert G[0].tolist() == [7 * H] * P


def test_lpt_against_plain_python_and_bruteforce():
    rng = np.random.default_rng(3)
    for trial in range(60):
        P = int(rng.choice([2, 3, 4]))
        H = int(rng.choice([1, 2, 3]))
        E = P * H
        Le = rng.integers(0, 50, E).astype(np.int64)
        if trial % 3 == 0:
            Le[rng.integers(0, E, E // 2)] = Le[0]        # force ties
        pi, G = oracle.lpt(Le[None, :], P)
        pi, G = pi[0], G[0]
        # permutation onto slots, H per rank, loads add up
        assert sorted(pi.tolist()) == list(range(E))
        owner = pi // H
        assert np.bincount(owner, minlength=P).tolist() == [H] * P
        assert [int(Le[owner == p].sum()) for p in range(P)] == G.tolist()
        # the same greedy written with sorted() and min()
        load, cnt, want = [0] * P, [0] * P, {}
        for e in sorted(range(E), key=lambda e: (-int(Le[e]), e)):
            p = min((p for p in range(P) if cnt[p] < H), key=lambda p: (load[p], p))
            want[e] = p * H + cnt[p]
            load[p] += int(Le[e])
            cnt[p] += 1
        assert pi.tolist() == [want[e] for e in range(E)]
        # never better than the true optimum over all H-per-rank assignments
        if E <= 8:
            best = min(max(sum(int(Le[e]) for e in range(E) if asg[e] == p) for p in range(P))
                       for asg in itertools.product(range(P), repeat=E)
                       if all(asg.count(p) == H for p in range(P)))
            assert best <= G.max() <= 2 * best + 1


def test_projection_conservation_and_invariance():
    """Eq. physical-rank-demand, Eq. aggregate-invariance, Eq. packing-lower-bound."""
    w = hetero_window()
    s = w.spec
    pi, G, q = placed(w)
    assert oracle.check_window(w.lengths, w.demand, s.top_k, s.token_cap) == 0
    assert (q.sum(axis=2) == s.top_k * w.lengths[:, None]).all()
    assert (q.sum(axis=0) == G).all()
    onehot = np.zeros((s.n_layers, s.n_experts, s.ep_width), np.int64)
    for l in range(s.n_layers):
        onehot[l, np.arange(s.n_experts), pi[l] // (s.n_experts // s.ep_width)] = 1
    assert (np.einsum("ile,lep->ilp", w.demand.astype(np.int64), onehot) == q).all()
    R, cert, seed = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width)
    rng = np.random.default_rng(4)
    for edp in (None, [0, 0, 1, 1], [0, 0, 0, 0]):
        for _ in range(3):
            lay = rng.integers(0, R * s.dp_width, s.n_samples).astype(np.int32)
            ev = oracle.eval_layouts(w.lengths, q, lay, R, s.token_cap, s.dp_width, edp)
            assert (ev["W"][0].sum(axis=(0, 1)) == G).all()
            assert (ev["W"][0].max(axis=3).sum(axis=(0, 1)) >= G.max(axis=1)).all()


def test_window_checks_reject_bad_input():
    w = hetero_window()
    s = w.spec
    bad = w.demand.copy()
    bad[5, 1, 2] += 1
    assert oracle.check_window(w.lengths, bad, s.top_k, s.token_cap) == 6
    t = w.lengths.copy()
    t[3] = s.token_cap + 1
    assert oracle.check_window(t, w.demand, s.top_k, s.token_cap) == 4


# ----------------------------------------------------------------------------------------
# objective
# ----------------------------------------------------------------------------------------
def test_uniform_routing_closed_form():
    """Eq. row-expert-cost with q = k*t/P on every rank: E[r][g] = L*k*T[r][g]/(P*C);
    with P = 1 it is L*k*Tbar."""
    rng = np.random.default_rng(5)
    N, L, k, C, D, R = 24, 3, 2, 4096, 2, 3
    for P in (1, 4):
        t = (rng.integers(1, 60, N) * P).astype(np.int32)
        q = np.repeat((k * t // P)[:, None, None], L, 1).repeat(P, 2).astype(np.int32)
        lay = (np.arange(N) % (R * D)).astype(np.int32)
        for edp in ([0, 1], [0, 0]):
            ev = oracle.eval_layouts(t, q, lay, R, C, D, edp)
            G = max(edp) + 1
            Trg = np.zeros((R, G), np.int64)
            for c in range(R * D):
                Trg[c // D, edp[c % D]] += ev["T"][0][c]
            assert (ev["Efx"][0] == 256 * C * (L * k * Trg // P)).all()


def test_pure_linear_attention_is_makespan():
    """No MoE layers' worth of load (q = 0) and beta = 0: s0 is the largest column token sum."""
    rng = np.random.default_rng(6)
    N, C, D, R = 30, 1000, 3, 2
    t = rng.integers(1, 90, N).astype(np.int32)
    q = np.zeros((N, 1, 1), np.int32)
    lay = rng.integers(0, R * D, N).astype(np.int32)
    ev = oracle.eval_layouts(t, q, lay, R, C, D, None, alpha=(1.0,), beta=(0.0,))
    col = np.zeros(D, np.int64)
    for i in range(N):
        col[lay[i] % D] += t[i]
    assert ev["score"][0][0] == 256 * C * col.max()
    assert ev["score"][0][1] == 256 * C * t.sum()


def test_integer_score_equals_real_valued_objective():
    w = hetero_window(N=60, L=4, E=16, k=2, C=4096, D=4, P=4, seed=11)
    s = w.spec
    _, _, q = placed(w)
    R, _, seed = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width)
    rng = np.random.default_rng(7)
    SC = oracle.score_scale(s.token_cap)
    for edp in (None, [0, 0, 1, 1], [0, 1, 0, 1], [0] * 4):
        for alpha, beta in (((1.0, 1.0), (0.0, 1.0)), ((0.5, 2.25, 1.0), (0.0, 0.75, 3.0))):
            lay = rng.integers(0, R * s.dp_width, s.n_samples).astype(np.int32)
            ev = oracle.eval_layouts(w.lengths, q, lay, R, s.token_cap, s.dp_width, edp, alpha, beta)
            real = oracle.eval_f64(w.lengths, q, lay, R, s.token_cap, s.dp_width, edp, alpha, beta)
            np.testing.assert_allclose(ev["score"][0] / SC, real, rtol=1e-12)
            mine = score_matrix_form(w.lengths, q, lay, R, s.dp_width, list(edp or range(4)),
                                     s.token_cap, alpha, beta)
            assert tuple(int(x) for x in ev["score"][0]) == mine


# ----------------------------------------------------------------------------------------
# row count and the length-only seed
# ----------------------------------------------------------------------------------------
def fits(t, K, C):
    """Exact: can the samples be split into K non-empty bins of capacity C? (tiny inputs)"""
    t = sorted(t, reverse=True)

    def go(i, bins, used):
        if i == len(t):
            return used == K
        if len(t) - i < K - used:
            return False
        seen = set()
        for b in range(used):
            if bins[b] + t[i] <= C and bins[b] not in seen:
                seen.add(bins[b])
                bins[b] += t[i]
                if go(i + 1, bins, used):
                    return True
                bins[b] -= t[i]
        if used < K:
            bins[used] = t[i]
            if go(i + 1, bins, used + 1):
                return True
            bins[used] = 0
        return False

    return go(0, [0] * K, 0)


def ffd_plain(t, K, C):
    """First-fit-decreasing into exactly K bins (Section 3.2 reading): the K longest samples open the
    bins, every later one goes to the lowest bin it fits in; None when some sample fits nowhere."""
    order = sorted(range(len(t)), key=lambda i: (-t[i], i))
    if K > len(t):
        return None
    fill = [t[i] for i in order[:K]]
    if any(f > C for f in fill):
        return None
    for i in order[K:]:
        b = next((b for b in range(K) if fill[b] + t[i] <= C), None)
        if b is None:
            return None
        fill[b] += t[i]
    return fill


def test_pack_ffd_properties_and_certificate():
    rng = np.random.default_rng(8)
    for trial in range(40):
        N, D, C = int(rng.integers(4, 12)), int(rng.choice([1, 2, 3])), 100
        t = rng.integers(5, 90, N).astype(np.int32)
        R, cert, cell = oracle.pack_ffd(t, C, D)
        if R == 0:      # no row count packs: the plain first-fit-decreasing below fails for every one of them
            assert all(ffd_plain(t.tolist(), r * D, C) is None for r in range(1, N // D + 1))
            continue
        assert ffd_plain(t.tolist(), R * D, C) is not None
        assert all(ffd_plain(t.tolist(), r * D, C) is None for r in range(max(1, -(-int(t.sum()) // (C * D))), R))
        K = R * D
        fill = np.bincount(cell, weights=t, minlength=K)
        assert K <= N and (fill <= C).all() and (np.bincount(cell, minlength=K) >= 1).all()
        assert R >= -(-int(t.sum()) // (C * D))
        if cert:    # certified minimal: one row fewer is impossible
            assert R == 1 or not fits(t.tolist(), (R - 1) * D, C)
        assert fits(t.tolist(), K, C)
    # min_rows is a lower bound on R (pipeline occupancy, Section 3.2)
    t = np.full(12, 10, np.int32)
    assert oracle.pack_ffd(t, 100, 2)[0] == 1
    assert oracle.pack_ffd(t, 100, 2, min_rows=3)[0] == 3
    # infeasible: a sample longer than the cap, fewer samples than slots
    assert oracle.pack_ffd(np.array([5, 200], np.int32), 100, 1)[0] == 0
    assert oracle.pack_ffd(np.array([5], np.int32), 100, 2)[0] == 0


# ----------------------------------------------------------------------------------------
# resampling
# ----------------------------------------------------------------------------------------
def test_resampling_special_cases():
    SC = oracle.score_scale(4096)
    cq = int(oracle.schedule(2, 1e-3, 0.5)[1][0])
    rng = np.random.default_rng(9)
    P = 64
    for x in rng.integers(0, 2 ** 32, 20):
        # equal energies: everyone survives once
        assert oracle.resample(np.full(P, 50 * SC), SC, cq, int(x)).tolist() == list(range(P))
        # one member far below the rest: it takes every slot
        e = np.full(P, 80 * SC)
        e[17] = 40 * SC
        assert oracle.resample(e, SC, cq, int(x)).tolist() == [17] * P
        # general: ancestors ascend, offspring counts are floor or ceil of P*w/sum(w)
        e = (50 * SC * (1 + 2e-4 * rng.random(P))).astype(np.int64)
        anc = oracle.resample(e, SC, cq, int(x))
        assert (np.diff(anc) >= 0).all()
        emin = int(e.min())
        wts = np.array([oracle.exp2neg(min(2 ** 40, (min(2 ** 48 - 1, ((int(v) - emin) << 32) // emin) * cq) >> 16))
                        for v in e], dtype=np.float64)
        expect = P * wts / wts.sum()
        counts = np.bincount(anc, minlength=P)
        assert (counts >= np.floor(expect) - 1e-9).all() and (counts <= np.ceil(expect) + 1e-9).all()


def test_resampling_weights_follow_boltzmann():
    """w_j proportional to exp(-(1/T' - 1/T) * Etilde_j) (Algorithm 3)."""
    SC = oracle.score_scale(4096)
    T, ratio = 1e-3, 0.5
    cq = int(oracle.schedule(2, T, ratio)[1][0])
    P = 4096
    e = np.full(P, 60 * SC, np.int64)
    e[P // 2:] += int(60 * SC * 0.0007)             # Etilde = 7e-4 for the upper half
    want_ratio = math.exp(-(1 / (T * ratio) - 1 / T) * 0.0007)
    anc = oracle.resample(e, SC, cq, 12345)
    upper = (anc >= P // 2).sum()
    got_ratio = upper / (P - upper)
    assert abs(got_ratio - want_ratio) < 0.01


# ----------------------------------------------------------------------------------------
# annealing
# ----------------------------------------------------------------------------------------
def run(w, q, R, init, edp=None, **kw):
    s = w.spec
    args = dict(n_levels=6, steps=40, t0=s.t0, t_ratio=0.5, p_reloc=s.p_reloc, p_guide=s.p_guide,
                seed=3, edp_of_dp=edp, alpha=s.alpha, beta=s.beta)
    args.update(kw)
    return oracle.anneal(w.lengths, q, init, R, s.token_cap, s.dp_width, **args)


@pytest.mark.parametrize("edp", [None, [0, 0, 1, 1], [0, 0, 0, 0]])
def test_incremental_score_equals_full_rescoring(edp):
    """Section 4.1.2: IncrementalScore is equivalent to rescoring from scratch, so the whole
    trajectory (every accept decision, every ancestor) must be the same either way."""
    w = hetero_window()
    _, _, q = placed(w)
    R, _, seed = oracle.pack_ffd(w.lengths, w.spec.token_cap, w.spec.dp_width, min_rows=3)
    init = np.tile(seed, (6, 1))
    a = run(w, q, R, init, edp)
    b = run(w, q, R, init, edp, full_rescore=True)
    assert a["status"] == 0 and b["status"] == 0
    for key in ("term", "best", "best_step", "digest", "anc", "incumbent", "best_layout", "final_pop", "counters"):
        assert (a[key] == b[key]).all(), key
    assert a["counters"][2] > 100         # moves were accepted, so this compares something


def test_annealing_keeps_the_feasible_set_and_never_regresses():
    """Section 3.6: proposals keep coverage, capacity, non-empty cells, row count and topology;
    the returned plan is no worse than the best seed."""
    w = hetero_window(N=64, D=4, seed=21)
    s = w.spec
    _, _, q = placed(w)
    R, _, seed = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width, min_rows=3)
    init = np.tile(seed, (8, 1))
    res = run(w, q, R, init, [0, 0, 1, 1], n_levels=8, steps=60)
    assert res["status"] == 0
    K = R * s.dp_width
    for lay in list(res["final_pop"]) + [res["best_layout"]]:
        assert lay.min() >= 0 and lay.max() < K
        assert (np.bincount(lay, minlength=K) >= 1).all()
        assert (np.bincount(lay, weights=w.lengths, minlength=K) <= s.token_cap).all()
    seed_score = oracle.eval_layouts(w.lengths, q, seed, R, s.token_cap, s.dp_width, [0, 0, 1, 1])["score"][0]
    assert tuple(res["best_score"]) <= tuple(seed_score)
    # incumbent is monotone over levels and equals its own rescoring
    inc = [tuple(x) for x in res["incumbent"]]
    assert all(b <= a for a, b in zip(inc, inc[1:]))
    again = oracle.eval_layouts(w.lengths, q, res["best_layout"], R, s.token_cap, s.dp_width, [0, 0, 1, 1])["score"][0]
    assert tuple(again) == tuple(res["best_score"]) == inc[-1]
    # trajectory-best is never worse than the terminal state, and best_step = 0 means "start"
    assert all(tuple(b) <= tuple(t_) for b, t_ in zip(res["best"].reshape(-1, 3), res["term"].reshape(-1, 3)))


# ----------------------------------------------------------------------------------------
# GuidedProposal (Section 4.1.2) and the search energy (Eq. pa-energy)
# ----------------------------------------------------------------------------------------
def word_for(index, n):
    """Smallest 32-bit word x with floor(x * n / 2^32) == index."""
    return (index * 2 ** 32 + n - 1) // n


def proposal_fixture(edp=None, seed=7, alpha=(1.0, 1.0), beta=(0.0, 1.0)):
    """A heterogeneous window on 3 rows x 4 slots with, per cell, the row-shard cost J, its
    attention part A and the cell's own attention cost, all in plain Python integers."""
    w = make_window(custom_spec("prop", 48, 3, 8, 2, 2048, 4, 4, 4, 100, data_seed=seed, alpha=alpha, beta=beta))
    s = w.spec
    _, _, q = placed(w)
    R, _, lay = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width, min_rows=3)
    D, C = s.dp_width, s.token_cap
    shard = list(range(D)) if edp is None else list(edp)
    t = [int(x) for x in w.lengths]
    ah = [int(math.floor(a * 256 + 0.5)) for a in alpha]
    bh = [int(math.floor(b * 256 + 0.5)) for b in beta]
    K = R * D
    T = [sum(t[i] for i in range(len(t)) if lay[i] == c) for c in range(K)]
    Q = [sum(t[i] ** 2 for i in range(len(t)) if lay[i] == c) for c in range(K)]
    att = [sum(ah[x] * C * T[c] + bh[x] * Q[c] for x in range(len(ah))) for c in range(K)]
    Jc, Ac = [0] * K, [0] * K
    for c in range(K):
        r, g = c // D, shard[c % D]
        cells = [r * D + d for d in range(D) if shard[d] == g]
        A = sum(max(ah[x] * C * T[k] + bh[x] * Q[k] for k in cells) for x in range(len(ah)))
        Wsum = np.asarray(q, dtype=object)[[i for i in range(len(t)) if lay[i] in cells]].sum(axis=0)
        Jc[c] = A + 256 * C * sum(int(max(row)) for row in Wsum)
        Ac[c] = A
    return dict(w=w, q=q, R=R, lay=lay, K=K, N=len(t), J=Jc, A=Ac, att=att, edp=edp, alpha=alpha, beta=beta)


def propose(fx, A, B, rho=0.25, guide=0.8):
    s = fx["w"].spec
    return oracle.propose_once(fx["w"].lengths, fx["q"], fx["lay"], fx["R"], s.token_cap, s.dp_width, A, B,
                               int(math.floor(rho * 2 ** 32)), int(math.floor(guide * 2 ** 32)), fx["edp"],
                               fx["alpha"], fx["beta"])[0]


def test_guided_proposal_thresholds_and_branches():
    """Which word decides what: relocation iff A0 < rho*2^32, guided iff A1 < p_guide*2^32 (the
    paper's 0.8), the uniform branch reads A2, A3 only, the guided branch takes its targets from B0, B1."""
    fx = proposal_fixture()
    N, K, lay = fx["N"], fx["K"], fx["lay"]
    rho_q, guide_q = int(math.floor(0.25 * 2 ** 32)), int(math.floor(0.8 * 2 ** 32))
    a2, a3, b0, b1 = word_for(5, N), word_for(17, N), word_for(30, N), word_for(41, N)
    # uniform swap: sample pick(A2), partner pick(A3); the B words change nothing
    for B in ([b0, b1, 0, 0], [1, 2 ** 32 - 1, 2 ** 31, 7]):
        mv = propose(fx, [rho_q, guide_q, a2, a3], B)
        assert mv == dict(reloc=0, i=5, i2=17, c1=int(lay[5]), c2=int(lay[17]))
    # one below the relocation threshold: the same words now relocate sample 5 to cell pick(A3, K)
    mv = propose(fx, [rho_q - 1, guide_q, a2, word_for(9, K)], [b0, b1, 0, 0])
    assert mv == dict(reloc=1, i=5, i2=-1, c1=int(lay[5]), c2=9)
    assert propose(fx, [rho_q, guide_q, a2, word_for(9, K)], [b0, b1, 0, 0])["reloc"] == 0
    # one below the guide threshold: sources {pick(A2), pick(A3)}, targets {pick(B0), pick(B1)}
    mv = propose(fx, [rho_q, guide_q - 1, a2, a3], [b0, b1, 2 ** 32 - 1, 0])
    assert mv["reloc"] == 0 and mv["i"] in (5, 17) and mv["i2"] in (30, 41)
    mv = propose(fx, [0, guide_q - 1, a2, a3], [word_for(2, K), word_for(10, K), 2 ** 32 - 1, 0])
    assert mv["reloc"] == 1 and mv["i"] in (5, 17) and mv["c2"] in (2, 10) and mv["i2"] == -1
    # rho = 0 never relocates, rho = 1 (threshold 2^32) always does; the same for p_guide
    assert propose(fx, [0, 0, a2, a3], [b0, b1, 0, 0], rho=0.0, guide=0.0) == dict(reloc=0, i=5, i2=17, c1=int(lay[5]), c2=int(lay[17]))
    assert propose(fx, [2 ** 32 - 1, 2 ** 32 - 1, a2, a3], [b0, b1, 2 ** 32 - 1, 0], rho=1.0, guide=1.0)["reloc"] == 1


@pytest.mark.parametrize("edp", [None, [0, 0, 1, 1]])
def test_guided_proposal_source_takes_the_larger_cost_and_target_the_smaller(edp):
    """Section 4.1.2: the source is biased to a row-shard with a large J, the target to a small one.
    Tournament of two on the row-shard cost (B2 = 2^32 - 1 keeps the attention key off): the larger
    key wins the source, the smaller the target, the first candidate on ties."""
    fx = proposal_fixture(edp)
    N, K, lay, J = fx["N"], fx["K"], fx["lay"], fx["J"]
    B2 = 2 ** 32 - 1
    assert all(B2 * J[c] >= fx["A"][c] << 32 for c in range(K))          # the coin never picks the attention key
    seen_first, seen_second = 0, 0
    for sa in range(0, N, 5):
        for sb in range(1, N, 7):
            ja, jb = J[lay[sa]], J[lay[sb]]
            src = sb if jb > ja else sa                                     # larger wins, tie -> first
            for ta, tb in ((3, 40), (40, 3), (11, 29), (22, 22)):
                want_t = tb if J[lay[tb]] < J[lay[ta]] else ta              # smaller wins, tie -> first
                mv = propose(fx, [2 ** 32 - 1, 0, word_for(sa, N), word_for(sb, N)],
                             [word_for(ta, N), word_for(tb, N), B2, 0])
                assert (mv["i"], mv["i2"]) == (src, want_t)
                assert (mv["c1"], mv["c2"]) == (int(lay[src]), int(lay[want_t]))
            for ca, cb in ((0, K - 1), (K - 1, 0), (4, 4), (2, 7)):         # relocation: target cells
                want_c = cb if J[cb] < J[ca] else ca
                mv = propose(fx, [0, 0, word_for(sa, N), word_for(sb, N)], [word_for(ca, K), word_for(cb, K), B2, 0])
                assert (mv["reloc"], mv["i"], mv["c2"]) == (1, src, want_c)
            seen_first += src == sa and ja != jb
            seen_second += src == sb
    assert seen_first > 5 and seen_second > 5                               # both outcomes were exercised
    # equal keys: two samples of one cell -> the first candidate
    same = [i for i in range(N) if lay[i] == lay[0]]
    assert len(same) >= 2
    mv = propose(fx, [2 ** 32 - 1, 0, word_for(same[1], N), word_for(same[0], N)], [word_for(3, N), word_for(40, N), B2, 0])
    assert mv["i"] == same[1]
    mv = propose(fx, [2 ** 32 - 1, 0, word_for(3, N), word_for(40, N)], [word_for(same[1], N), word_for(same[0], N), B2, 0])
    assert mv["i2"] == same[1]
    twins = [(a, b) for a in range(K) for b in range(K) if a != b and J[a] == J[b]]      # cells of one row-shard
    if twins:
        ca, cb = twins[-1]
        assert propose(fx, [0, 0, word_for(3, N), word_for(40, N)], [word_for(ca, K), word_for(cb, K), B2, 0])["c2"] == ca


def test_guided_proposal_attention_key_coin():
    """Section 4.1.2: the attention straggler is chosen in proportion to its contribution: the
    cell-attention key replaces the row-shard cost iff B2 * J < A * 2^32 for the first source
    candidate's row-shard (both sides of the boundary word), and then decides source and target."""
    fx = proposal_fixture()
    N, K, lay, J, A, att = fx["N"], fx["K"], fx["lay"], fx["J"], fx["A"], fx["att"]
    # a pair of samples on which the two keys disagree
    pair = next(((a, b) for a in range(N) for b in range(N)
                 if (J[lay[b]] > J[lay[a]]) != (att[lay[b]] > att[lay[a]]) and att[lay[a]] != att[lay[b]]
                 and J[lay[a]] != J[lay[b]]), None)
    assert pair is not None
    sa, sb = pair
    tpair = next(((a, b) for a in range(N) for b in range(N)
                  if (J[lay[b]] < J[lay[a]]) != (att[lay[b]] < att[lay[a]]) and att[lay[a]] != att[lay[b]]
                  and J[lay[a]] != J[lay[b]]), None)
    ta, tb = tpair
    ca = lay[sa]
    edge = -((-A[ca] << 32) // J[ca])              # smallest word with B2 * J >= A * 2^32
    assert 0 < edge < 2 ** 32
    by_J = (sb if J[lay[sb]] > J[lay[sa]] else sa, tb if J[lay[tb]] < J[lay[ta]] else ta)
    by_att = (sb if att[lay[sb]] > att[lay[sa]] else sa, tb if att[lay[tb]] < att[lay[ta]] else ta)
    assert by_J != by_att
    words = [2 ** 32 - 1, 0, word_for(sa, N), word_for(sb, N)]
    mv = propose(fx, words, [word_for(ta, N), word_for(tb, N), edge - 1, 0])
    assert (mv["i"], mv["i2"]) == by_att
    mv = propose(fx, words, [word_for(ta, N), word_for(tb, N), edge, 0])
    assert (mv["i"], mv["i2"]) == by_J
    # in proportion to its contribution: over uniform B2 the attention key is used with frequency A/J
    rng = np.random.default_rng(4)
    n = 4000
    hits = sum(propose(fx, words, [word_for(ta, N), word_for(tb, N), int(x), 0])["i"] == by_att[0]
               for x in rng.integers(0, 2 ** 32, n))
    pr = A[ca] / J[ca]
    assert abs(hits / n - pr) < 4 * math.sqrt(pr * (1 - pr) / n) + 1e-3


def test_guided_proposal_statistics_over_philox_draws():
    """Section 4.1.2 over the chain's own random words (Philox, purposes 0 and 1): 80 % of the
    proposals are guided, a quarter are relocations, sources sit in costlier row-shards than the
    average sample, targets in cheaper ones."""
    fx = proposal_fixture(alpha=(0.0, 0.0), beta=(0.0, 0.0))       # no attention cost: the key is always J
    N, K, lay, J = fx["N"], fx["K"], fx["lay"], fx["J"]
    assert len(set(J)) > 4
    n = 20000
    key = np.array([0x1234, 0x9], np.uint32)
    guided = reloc = larger = differ = 0
    src_J, dst_J = 0, 0
    for k in range(n):
        A = oracle.philox4x32_10([k, 3, 1, 0], key)
        B = oracle.philox4x32_10([k, 3, 1, 1], key)
        mv = propose(fx, A, B)
        sa, sb = int(A[2]) * N >> 32, int(A[3]) * N >> 32
        reloc += mv["reloc"]
        guided += int(A[1]) < int(math.floor(0.8 * 2 ** 32))
        if J[lay[sa]] != J[lay[sb]]:
            differ += 1
            larger += J[lay[mv["i"]]] == max(J[lay[sa]], J[lay[sb]])
        src_J += J[mv["c1"]]
        dst_J += J[mv["c2"]]
    sig = lambda p, m: 3.5 * math.sqrt(p * (1 - p) / m)
    assert abs(guided / n - 0.8) < sig(0.8, n)
    assert abs(reloc / n - 0.25) < sig(0.25, n)
    # the source holds the larger cost always when guided, half of the time otherwise: 0.8 + 0.2/2
    assert abs(larger / differ - 0.9) < sig(0.9, differ)
    mean_J = sum(J[lay[i]] for i in range(N)) / N
    assert src_J / n > mean_J > dst_J / n


def test_energy_coefficients():
    """Eq. pa-energy: E = s0 + 1e-6 * s1 + 1e-9 * s2, floored per term in integer units."""
    s0 = 123456789012
    assert oracle.energy([s0, 999999, 10 ** 9 - 1]) == s0
    assert oracle.energy([s0, 1000000, 10 ** 9 - 1]) == s0 + 1
    assert oracle.energy([s0, 999999, 10 ** 9]) == s0 + 1
    assert oracle.energy([s0, 7 * 10 ** 6 + 5, 3 * 10 ** 9 + 999]) == s0 + 10
    # equal s0: a difference of 10^6 in s1 weighs exactly what 10^9 in s2 does, and 1 in s0
    assert oracle.energy([s0, 2 * 10 ** 6, 0]) == oracle.energy([s0, 0, 2 * 10 ** 9]) == oracle.energy([s0 + 2, 0, 0])
    # and the chain ranks by it: at zero temperature a move that raises the energy is never kept
    big = (2 ** 40, 5 * 10 ** 15, 3 * 10 ** 12)
    assert oracle.energy(big) == 2 ** 40 + 5 * 10 ** 9 + 3000


def test_zero_temperature_only_descends():
    w = hetero_window(seed=5)
    _, _, q = placed(w)
    R, _, seed = oracle.pack_ffd(w.lengths, w.spec.token_cap, w.spec.dp_width, min_rows=2)
    res = run(w, q, R, np.tile(seed, (1, 1)), None, n_levels=5, steps=80, t0=1e-300, t_ratio=1.0)
    e = [int(s[0] + s[1] // 10 ** 6 + s[2] // 10 ** 9) for s in res["term"][:, 0]]
    assert all(b <= a for a, b in zip(e, e[1:]))
    assert (res["best"] == res["term"]).all()      # a descending chain ends on its best


def test_annealing_reaches_bruteforce_optimum_on_a_tiny_window():
    """8 samples, 2 rows x 2 DP slots: all 4^8 layouts can be scored; annealing must never
    beat the optimum and must find it with a modest budget."""
    w = make_window(custom_spec("bf", 8, 2, 4, 2, 512, 2, 2, 16, 100, data_seed=2))
    s = w.spec
    _, _, q = placed(w)
    R = 2
    t = w.lengths.astype(np.int64)
    best = None
    for code in range(4 ** 8):
        lay = [(code >> (2 * i)) & 3 for i in range(8)]
        fill = np.bincount(lay, weights=t, minlength=4)
        if (np.bincount(lay, minlength=4) == 0).any() or (fill > s.token_cap).any():
            continue
        sc = score_matrix_form(t, q, lay, R, 2, [0, 1], s.token_cap)
        if best is None or sc < best:
            best = sc
    seed = np.array([0, 1, 2, 3, 0, 1, 2, 3], np.int32)
    if (np.bincount(seed, weights=t, minlength=4) > s.token_cap).any():
        pytest.skip("seed layout infeasible for this draw")
    res = run(w, q, R, np.tile(seed, (16, 1)), None, n_levels=10, steps=100, t0=1e-2, t_ratio=0.5)
    assert res["status"] == 0
    assert tuple(int(x) for x in res["best_score"]) >= best
    assert tuple(int(x) for x in res["best_score"]) == best


def test_named_tiny_window_end_to_end():
    w = make_window("tiny")
    res = oracle.plan(w)
    assert res["status"] == 0 and res["n_rows"] >= 13
    assert res["counters"][0] == 8 * 200
    assert res["counters"][1] <= res["counters"][0] and res["counters"][2] <= res["counters"][1]


# ----------------------------------------------------------------------------------------
# diagnostics (Section 5.2: Eq. global-ep-cv, EP peak sum, tail peak, Eq. ep-efficiency)
# ----------------------------------------------------------------------------------------
def test_diagnostics_on_the_fig2_instance():
    """Window loads 12/4 -> mean 8, deviation 4, CV 0.5; after the permutation 8/8 -> CV 0.
    Packing A (row peaks 8, 8): S_EP 16, T_EP 8, each row's mean rank load is 4 -> eta 0.5.
    Packing B (row peaks 4, 4): S_EP 8, T_EP 4, eta 1."""
    a, m = read_fig2()
    Lagg = oracle.aggregate(a)
    pi, _ = oracle.lpt(Lagg, 2)
    q = oracle.project(a, pi, 2)
    t = np.full(4, 4, np.int32)
    dA = oracle.diagnostics(t, q, Lagg, pi, np.array(m["packing_A_rows"], np.int32), R=2, C_cap=8, D=1)
    dB = oracle.diagnostics(t, q, Lagg, pi, np.array(m["packing_B_rows"], np.int32), R=2, C_cap=8, D=1)
    assert dA["cv_identity"] == 0.5 and dA["cv_placed"] == 0.0
    assert (dA["s_ep"], dA["t_ep"], dA["eta_ep"]) == (16, 8, 0.5)
    assert (dB["s_ep"], dB["t_ep"], dB["eta_ep"]) == (8, 4, 1.0)
    assert dA["attention"] == 5.0 and dA["joint"] == 7.0 and dB["joint"] == 6.0


def test_diagnostics_against_numpy_and_placement_effect():
    w = hetero_window(N=80, L=4, E=16, k=2, C=4096, D=4, P=4, seed=31)
    s = w.spec
    Lagg = oracle.aggregate(w.demand)
    pi, G, q = placed(w)
    R, _, seed = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width, min_rows=3)
    edp = [0, 0, 1, 1]
    d = oracle.diagnostics(w.lengths, q, Lagg, pi, seed, R, s.token_cap, s.dp_width, edp)
    ev = oracle.eval_layouts(w.lengths, q, seed, R, s.token_cap, s.dp_width, edp)
    W = ev["W"][0].astype(np.int64)                      # [R][G][L][P]
    assert d["s_ep"] == W.max(axis=(1, 3)).sum() and d["t_ep"] == W.max()
    assert d["n_ep"] == W.sum(axis=3).max(axis=1).sum()
    assert abs(d["eta_ep"] - d["n_ep"] / (s.ep_width * d["s_ep"])) < 1e-15 and 0 < d["eta_ep"] <= 1
    Gf = G.astype(np.float64)
    want = np.mean(Gf.std(axis=1) / Gf.mean(axis=1))
    assert abs(d["cv_placed"] - want) < 1e-12
    assert d["cv_placed"] < d["cv_identity"]             # LPT lowers the aggregate skew
    SC = oracle.score_scale(s.token_cap)
    assert abs(d["attention"] - ev["Afx"][0].sum() / SC) < 1e-12 and abs(d["joint"] - ev["score"][0][0] / SC) < 1e-12


# ----------------------------------------------------------------------------------------
# randomized fixed-row seeds (Algorithm 2, trial loop)
# ----------------------------------------------------------------------------------------
def test_seed_trials_are_feasible_partitions_and_width_one_is_best_fit_decreasing():
    w = hetero_window(N=90, L=2, E=8, k=1, C=4096, D=3, P=4, seed=41)
    s = w.spec
    t = w.lengths
    R, _, seed = oracle.pack_ffd(t, s.token_cap, s.dp_width, min_rows=3)
    K = R * s.dp_width
    for width in (1, 4, 16):
        lays, ok = oracle.seed_trials(t, seed, R, s.token_cap, s.dp_width, 24, width, seed=9)
        assert ok[0] == 1 and (lays[0] == seed).all()
        for j in range(24):
            assert lays[j].min() >= 0 and lays[j].max() < K
            assert (np.bincount(lays[j], minlength=K) >= 1).all()
            assert (np.bincount(lays[j], weights=t, minlength=K) <= s.token_cap).all()
            if not ok[j]:
                assert (lays[j] == seed).all()
        if width == 1:
            # no randomness left: decreasing order, K longest open the cells, then the fullest
            # feasible cell (ties: fewer samples, lower index) -- plain best-fit-decreasing
            order = sorted(range(len(t)), key=lambda i: (-int(t[i]), i))
            fill, cnt, want = [0] * K, [0] * K, [0] * len(t)
            for h, i in enumerate(order):
                if h < K:
                    b = h
                else:
                    feas = [c for c in range(K) if fill[c] + t[i] <= s.token_cap]
                    b = min(feas, key=lambda c: (-fill[c], cnt[c], c))
                fill[b] += int(t[i]); cnt[b] += 1; want[i] = b
            assert ok[1:].all() and all((lays[j] == want).all() for j in range(1, 24))
        else:
            assert len({lays[j].tobytes() for j in range(24)}) > 12      # the trials really differ


def test_seed_trial_draws_are_uniform_over_the_window():
    """With as many cells as samples every sample opens the cell of its emission position, so the
    layout is the shuffle itself: the first emitted sample must be a uniform pick among the first
    w samples of the sorted order, and no sample can be emitted more than w-1 places early."""
    N, width = 64, 8
    t = np.full(N, 10, np.int32)                       # equal lengths: sorted order = index order
    seed = np.arange(N, dtype=np.int32)
    lays, ok = oracle.seed_trials(t, seed, 16, 10, 4, 4000, width, seed=5)
    assert ok.all()
    first = np.array([int(np.where(lays[j] == 0)[0][0]) for j in range(1, 4000)])
    counts = np.bincount(first, minlength=N)
    assert counts[width:].sum() == 0
    assert abs(counts[:width] - 3999 / width).max() < 5 * (3999 / width * (1 - 1 / width)) ** 0.5
    for j in range(1, 200):
        assert sorted(lays[j].tolist()) == list(range(N))            # a permutation
        assert (lays[j] >= np.arange(N) - (width - 1)).all()         # sample i leaves no earlier than i-(w-1)


# ---- EDPAwarePair (Section 4.1.1, Algorithm 2) ---------------------------------------------
def _pair_inputs(profiles):
    """One sample per cell whose demand row is the given profile [K][L][P]."""
    prof = np.asarray(profiles, np.int32)
    K = prof.shape[0]
    q = prof.copy()
    lay = np.arange(K, dtype=np.int32)
    return q, lay


def test_edp_pair_worked_example_balances_the_shared_shard():
    """Two rows of two DP slots that share one EDP shard; one layer, two ranks.  Cells a, c load
    rank 0 with 10 tokens, cells b, d load rank 1.  Greedy pairing (width 1): a opens row 0; b adds
    nothing to the peak sum of row 0 (key (0, 10)) but 10 to row 1, so it joins a; c then only has
    row 1 left, d follows.  Rows {a, b}, {c, d}: each row peaks at 10 instead of 20 for {a, c}."""
    prof = [[[10, 0]], [[0, 10]], [[10, 0]], [[0, 10]]]
    q, lay = _pair_inputs(prof)
    pop = np.stack([lay, lay])
    out = oracle.edp_pair(q, pop, R=2, D=2, width=1, seed=3, edp_of_dp=[0, 0])
    assert (out[0] == lay).all()                     # member 0 is never touched
    assert out[1].tolist() == [0, 1, 2, 3]
    # same cells listed as a, c, b, d: the pairing must undo the bad order (a with b, c with d)
    prof2 = [prof[0], prof[2], prof[1], prof[3]]
    q2, lay2 = _pair_inputs(prof2)
    out2 = oracle.edp_pair(q2, np.stack([lay2, lay2]), R=2, D=2, width=1, seed=3, edp_of_dp=[0, 0])
    rows = out2[1] // 2
    assert rows[0] == rows[2] and rows[1] == rows[3] and rows[0] != rows[1]


def test_edp_pair_second_key_breaks_equal_increases():
    """One shard, two rows of two slots, two layers, one rank.  a = (10, 0) opens row 0.  b = (0, 8)
    raises the peak sum by 8 in either row, but the largest peak would be 10 in row 0 and 8 in row 1:
    the second key sends it to row 1 (slot 2) although slot 1 has the lower index.  c = (1, 0) adds 1
    anywhere; the peak is 11 beside a and 8 beside b, so it joins b (slot 3); d = (0, 1) takes slot 1."""
    prof = [[[10], [0]], [[0], [8]], [[1], [0]], [[0], [1]]]
    q, lay = _pair_inputs(prof)
    out = oracle.edp_pair(q, np.stack([lay, lay]), R=2, D=2, width=1, seed=11, edp_of_dp=[0, 0])
    assert out[1].tolist() == [0, 2, 3, 1]


def test_edp_pair_identity_shards_sorts_cells_by_peak():
    """With one shard per DP slot every empty slot has an empty row-shard, so all keys tie and the
    lowest slot wins: greedy pairing lists the cells by decreasing peak (ties: lower index)."""
    rng = np.random.default_rng(4)
    K, L, P = 12, 3, 4
    prof = rng.integers(0, 50, (K, L, P))
    prof[5] = prof[2]                                   # a tie
    q, lay = _pair_inputs(prof)
    out = oracle.edp_pair(q, np.stack([lay, lay]), R=3, D=4, width=1, seed=1)
    peaks = prof.reshape(K, -1).max(1)
    order = sorted(range(K), key=lambda b: (-int(peaks[b]), b))
    want = np.empty(K, np.int64)
    for h, b in enumerate(order):
        want[b] = h
    assert out[1].tolist() == want.tolist()


def test_edp_pair_keeps_cells_and_its_greedy_step_is_the_smallest_key():
    w = hetero_window(N=80, L=3, E=8, k=2, C=4096, D=4, P=4, seed=17)
    s, t = w.spec, w.lengths
    edp = [0, 0, 1, 1]
    pi, _ = oracle.lpt(oracle.aggregate(w.demand), s.ep_width)
    q = oracle.project(w.demand, pi, s.ep_width)
    R, _, seed_lay = oracle.pack_ffd(t, s.token_cap, s.dp_width, min_rows=3)
    K = R * s.dp_width
    lays, ok = oracle.seed_trials(t, seed_lay, R, s.token_cap, s.dp_width, 16, 4, seed=9)
    for width in (1, 3):
        out = oracle.edp_pair(q, lays, R, s.dp_width, width, seed=9, edp_of_dp=edp)
        assert (out[0] == lays[0]).all()
        for j in range(1, 16):
            # a bijection of cells onto slots: samples that shared a cell still do, nothing else does
            m = {}
            for i in range(len(t)):
                assert m.setdefault(int(lays[j][i]), int(out[j][i])) == int(out[j][i])
            assert sorted(m.values()) == sorted(set(m.values())) and len(m) == K
    # width 1, member 1: replay the greedy rule with plain numpy and compare slot by slot
    out = oracle.edp_pair(q, lays, R, s.dp_width, 1, seed=9, edp_of_dp=edp)
    lay = lays[1]
    prof = np.zeros((K,) + q.shape[1:], np.int64)
    np.add.at(prof, lay, q)
    V = np.zeros((R, 2) + q.shape[1:], np.int64)
    empty = [True] * K
    slot_of = {}
    for b in sorted(range(K), key=lambda b: (-int(prof[b].max()), b)):
        best = None
        for sl in range(K):
            if not empty[sl]:
                continue
            v = V[sl // 4, edp[sl % 4]]
            key = (int((v + prof[b]).max(1).sum() - v.max(1).sum()), int((v + prof[b]).max()), sl)
            if best is None or key < best:
                best = key
        sl = best[2]
        empty[sl] = False
        slot_of[b] = sl
        V[sl // 4, edp[sl % 4]] += prof[b]
    assert [slot_of[int(b)] for b in lay] == out[1].tolist()


def test_edp_pair_sampling_ranks_decay_by_halves():
    """Identity shards, so the ranking of the empty slots is the slot order itself and the cell with
    the largest peak lands on slot rho of the first draw: rho = 0, 1, 2 with probability 1/2, 1/4 and
    (width 3) the remaining 1/4."""
    K, L, P = 6, 1, 2
    prof = np.zeros((K, L, P), np.int64)
    prof[:, 0, 0] = [60, 50, 40, 30, 20, 10]
    q, lay = _pair_inputs(prof)
    n = 4001
    out = oracle.edp_pair(q, np.tile(lay, (n, 1)), R=2, D=3, width=3, seed=77)
    first = out[1:, 0]                                   # slot of the cell with the largest peak
    freq = np.bincount(first, minlength=K) / (n - 1)
    assert freq[3:].sum() == 0
    assert abs(freq[0] - 0.5) < 0.03 and abs(freq[1] - 0.25) < 0.03 and abs(freq[2] - 0.25) < 0.03


# ---- Canonicalize / CanonicalMap / QualityDiversitySelect (Section 4.1.1) -------------------
def _small_population(seed=23, pop=20, edp=(0, 0, 1, 1)):
    w = hetero_window(N=60, L=3, E=8, k=2, C=4096, D=4, P=4, seed=seed)
    s, t = w.spec, w.lengths
    pi, _ = oracle.lpt(oracle.aggregate(w.demand), s.ep_width)
    q = oracle.project(w.demand, pi, s.ep_width)
    R, _, seed_lay = oracle.pack_ffd(t, s.token_cap, s.dp_width, min_rows=3)
    lays, _ = oracle.seed_trials(t, seed_lay, R, s.token_cap, s.dp_width, pop, 4, seed=9)
    return w, q, R, lays, list(edp)


def test_canonicalize_by_hand_and_its_symmetries():
    # two rows of two exchangeable slots; cells {0,4} {1,5} in row 1 and {2} {3} in row 0, listed backwards
    assert oracle.canonicalize([3, 2, 1, 0, 3, 2], 2, 2, [0, 0]).tolist() == [0, 1, 2, 3, 0, 1]
    # slots of different shards are not exchangeable: only the rows are reordered
    assert oracle.canonicalize([3, 2, 1, 0, 3, 2], 2, 2, [0, 1]).tolist() == [1, 0, 3, 2, 1, 0]
    w, q, R, lays, edp = _small_population()
    s, t = w.spec, w.lengths
    D = s.dp_width
    rng = np.random.default_rng(1)
    for j in range(6):
        x = lays[j]
        cx = oracle.canonicalize(x, R, D, edp)
        assert (oracle.canonicalize(cx, R, D, edp) == cx).all()                   # idempotent
        # the canonical form is the same plan: same co-assignment, same score
        assert oracle.coassign_q20(x, cx) == 0 and oracle.coassign_q20(x // D, cx // D) == 0
        ex = oracle.eval_layouts(t, q, np.stack([x, cx]), R, s.token_cap, D, edp, s.alpha, s.beta)["score"]
        assert (ex[0] == ex[1]).all()
        # every row permutation combined with swaps inside the shards gives the same signature
        for _ in range(5):
            rows = rng.permutation(R)
            slot = np.arange(D)
            for g in set(edp):
                ds = [d for d in range(D) if edp[d] == g]
                slot[ds] = rng.permutation(ds)
            y = rows[x // D] * D + slot[x % D]
            assert (oracle.canonicalize(y, R, D, edp) == cx).all()
        # moving a cell across shards changes the plan, hence the signature
        y = (x // D) * D + np.array([2, 1, 0, 3])[x % D]
        assert (oracle.canonicalize(y, R, D, edp) != cx).any()


def test_coassignment_distance_special_cases():
    assert oracle.coassign_q20([0, 0, 1, 1], [0, 0, 0, 1]) == 786432        # 1 common pair of 4: 1 - 1/4
    assert oracle.coassign_q20([0, 0, 1, 1], [5, 5, 9, 9]) == 0             # same partition, other names
    assert oracle.coassign_q20([0, 0, 1, 1], [0, 1, 0, 1]) == 1 << 20       # no common pair
    assert oracle.coassign_q20([0, 1, 2, 3], [3, 2, 1, 0]) == 0             # nobody together in either
    rng = np.random.default_rng(3)
    a, b = rng.integers(0, 5, 40), rng.integers(0, 7, 40)
    assert oracle.coassign_q20(a, b) == oracle.coassign_q20(b, a)
    # against the contingency-table form of the same count
    tab = np.zeros((5, 7), np.int64)
    np.add.at(tab, (a, b), 1)
    both = int((tab * (tab - 1) // 2).sum())
    pa = int((tab.sum(1) * (tab.sum(1) - 1) // 2).sum())
    pb = int((tab.sum(0) * (tab.sum(0) - 1) // 2).sum())
    assert oracle.coassign_q20(a, b) == (1 << 20) - (both << 20) // (pa + pb - both)


def test_sketch_is_row_order_invariant_and_matches_a_plain_restatement():
    w, q, R, lays, edp = _small_population()
    s, t = w.spec, w.lengths
    D, nproj = s.dp_width, 5
    x = lays[3]
    phi = oracle.sw_sketch(t, q, x, R, s.token_cap, D, s.top_k, nproj, 77, edp)
    assert (np.diff(phi, axis=1) >= 0).all()
    rows = np.random.default_rng(2).permutation(R)
    y = rows[x // D] * D + x % D
    assert (oracle.sw_sketch(t, q, y, R, s.token_cap, D, s.top_k, nproj, 77, edp) == phi).all()
    # features and projections restated with numpy
    G, L = max(edp) + 1, q.shape[1]
    W = np.zeros((R, G, L, q.shape[2]), np.int64)
    np.add.at(W, (x // D, np.asarray(edp)[x % D]), q)
    Tr = np.bincount(x // D, weights=t, minlength=R).astype(np.int64)
    Qr = np.bincount(x // D, weights=t.astype(np.int64) ** 2, minlength=R).astype(np.int64)
    H = np.zeros((R, 2 + G * L), np.int64)
    H[:, 0] = (Tr << 16) // (s.token_cap * D)
    H[:, 1] = (Qr << 16) // (s.token_cap * s.token_cap * D)
    ng = np.bincount(edp, minlength=G)
    for g in range(G):
        H[:, 2 + g * L: 2 + (g + 1) * L] = (W[:, g].max(-1) << 16) // (s.top_k * s.token_cap * ng[g])
    for kk in range(nproj):
        sign = np.array([-1 if oracle.philox4x32_10((f, 0, kk, 7), (77, 0))[0] >> 31 else 1 for f in range(H.shape[1])])
        assert (np.sort(H @ sign) == phi[kk]).all()


def test_canonical_map_and_quality_diversity_selection():
    w, q, R, lays, edp = _small_population(pop=24)
    s, t = w.spec, w.lengths
    D = s.dp_width
    rng = np.random.default_rng(8)
    pop = lays.copy()
    # members 20..23 are disguised copies (row order and exchangeable slots changed) of members 3, 3, 7, 0
    for dst, src in ((20, 3), (21, 3), (22, 7), (23, 0)):
        rows = rng.permutation(R)
        pop[dst] = rows[lays[src] // D] * D + np.array([1, 0, 3, 2])[lays[src] % D]
    sc = oracle.eval_layouts(t, q, pop, R, s.token_cap, D, edp, s.alpha, s.beta)["score"]
    sig = [oracle.canonicalize(x, R, D, edp).tobytes() for x in pop]
    classes = {}
    for j, k in enumerate(sig):
        classes.setdefault(k, []).append(j)
    for eta in (0, 1 << 16, 1 << 26):
        out = oracle.select_population(t, q, pop, sc, R, s.token_cap, D, s.top_k, 6, eta, 5, edp, want_dist=True)
        nd, order, dist = out["n_distinct"], out["order"], out["dist"]
        assert nd == len(classes) <= 20
        # one representative per class: lowest score, then lowest index (a copy scores like its source)
        reps = sorted(min(js, key=lambda j: (tuple(sc[j]), j)) for js in classes.values())
        assert sorted(order[:nd].tolist()) == reps
        assert all(j < 20 for j in reps)
        # starts from the exact-score winner; members repeat cyclically once all are used
        assert order[0] == min(reps, key=lambda j: (tuple(sc[j]), j))
        assert (order[nd:] == np.resize(order[:nd], len(order))[nd:]).all()
        assert all((out["layouts"][m] == pop[order[m]]).all() for m in range(len(order)))
        # distances: symmetric, zero on the diagonal and between a plan and its disguised copy
        assert (dist == dist.T).all() and (np.diag(dist) == 0).all() and dist[20, 3] == 0 and dist[23, 0] == 0
        # every pick maximises (distance to the nearest selected - penalty) among the remaining ones
        s0 = int(sc[order[0]][0])
        pen = {j: ((((int(sc[j][0]) - s0) << 20) // s0) * eta) >> 16 for j in reps}
        chosen = [int(order[0])]
        for n in range(1, nd):
            rest = [j for j in reps if j not in chosen]
            val = {j: min(int(dist[j, y]) for y in chosen) - pen[j] for j in rest}
            top = max(val.values())
            assert int(order[n]) == min(j for j in rest if val[j] == top)
            chosen.append(int(order[n]))
    # a large eta turns the order into the score order (by primary score)
    prim = [int(sc[j][0]) for j in order[:nd]]
    assert prim == sorted(prim)
