"""ctypes loader for the plain C oracle (TEST INFRASTRUCTURE, not the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package.
It builds ``routepack_oracle.c`` with gcc on first use and exposes numpy-level wrappers
whose names follow the paper's notation.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "routepack_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_routepack.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, -O2, OpenMP for the per-chain loop)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True, text=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_nl2.restype = C.c_uint64
        _lib.orc_nl2.argtypes = [C.c_uint32]
        _lib.orc_exp2neg.restype = C.c_uint64
        _lib.orc_exp2neg.argtypes = [C.c_uint64]
        _lib.orc_check_window.restype = C.c_int64
        _lib.orc_pack_ffd.restype = C.c_int32
        _lib.orc_anneal.restype = C.c_int32
        _lib.orc_coassign_q20.restype = C.c_int64
        _lib.orc_accept_uphill.restype = C.c_int32
        _lib.orc_accept_uphill.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_uint64, C.c_uint32]
        _lib.orc_propose_once.restype = C.c_int32
        _lib.orc_energy.restype = C.c_int64
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


# ---- primitives -------------------------------------------------------------------------
def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def nl2(x: int) -> int:
    return int(lib().orc_nl2(int(x)))


def exp2neg(z: int) -> int:
    return int(lib().orc_exp2neg(int(z)))


def accept_uphill(e_old: int, e_new: int, SC: int, tau: int, x: int) -> bool:
    """The random part of the Metropolis test for an energy increase, given the accept word x."""
    return bool(lib().orc_accept_uphill(int(e_old), int(e_new), int(SC), int(tau), int(x)))


def exp2_table() -> np.ndarray:
    out = np.zeros(24, dtype=np.uint64)
    lib().orc_exp2_table(_p(out))
    return out


def schedule(n_levels: int, t0: float, t_ratio: float):
    tau = np.zeros(n_levels, dtype=np.uint64)
    cq = np.zeros(n_levels, dtype=np.uint64)
    lib().orc_schedule(C.c_int32(n_levels), C.c_double(t0), C.c_double(t_ratio), _p(tau), _p(cq))
    return tau, cq


def resample(energies: np.ndarray, SC: int, cq: int, x: int) -> np.ndarray:
    e = np.ascontiguousarray(energies, dtype=np.int64)
    anc = np.zeros(e.shape[0], dtype=np.int32)
    lib().orc_resample(C.c_int32(e.shape[0]), _p(e), C.c_int64(SC), C.c_uint64(cq), C.c_uint32(x), _p(anc))
    return anc


# ---- placement --------------------------------------------------------------------------
def check_window(lengths, demand, top_k: int, token_cap: int) -> int:
    t = _i32(lengths)
    a = _i32(demand)
    N, L, E = a.shape
    return int(lib().orc_check_window(C.c_int32(N), C.c_int32(L), C.c_int32(E), C.c_int32(top_k),
                                      C.c_int32(token_cap), _p(t), _p(a)))


def aggregate(demand) -> np.ndarray:
    a = _i32(demand)
    N, L, E = a.shape
    out = np.zeros((L, E), dtype=np.int64)
    lib().orc_aggregate(C.c_int32(N), C.c_int32(L), C.c_int32(E), _p(a), _p(out))
    return out


def lpt(Lagg: np.ndarray, P: int):
    """Algorithm 1 for every layer: returns (pi [L][E] slot ids, G [L][P] rank loads)."""
    Lagg = np.ascontiguousarray(Lagg, dtype=np.int64)
    L, E = Lagg.shape
    pi = np.zeros((L, E), dtype=np.int32)
    G = np.zeros((L, P), dtype=np.int64)
    for l in range(L):
        lib().orc_lpt_layer(C.c_int32(E), C.c_int32(P), _p(Lagg[l]), _p(pi[l]), _p(G[l]))
    return pi, G


def project(demand, pi, P: int) -> np.ndarray:
    a = _i32(demand)
    pi = _i32(pi)
    N, L, E = a.shape
    q = np.zeros((N, L, P), dtype=np.int32)
    lib().orc_project(C.c_int32(N), C.c_int32(L), C.c_int32(E), C.c_int32(P), _p(a), _p(pi), _p(q))
    return q


def pack_ffd(lengths, C_cap: int, D: int, min_rows: int = 0):
    """Row count and length-only seed: returns (R*, certified, cell_of [N]); R* = 0 if infeasible."""
    t = _i32(lengths)
    cell = np.zeros(t.shape[0], dtype=np.int32)
    cert = C.c_int32(0)
    R = lib().orc_pack_ffd(C.c_int32(t.shape[0]), C.c_int32(C_cap), C.c_int32(D), C.c_int32(min_rows),
                           _p(t), _p(cell), C.byref(cert))
    return int(R), int(cert.value), cell


def seed_trials(lengths, seed_layout, R: int, C_cap: int, D: int, pop_size: int, width: int, seed: int):
    """Randomized fixed-row seeds, one trial per member: returns (layouts [P][N], ok [P])."""
    t = _i32(lengths)
    sl = _i32(seed_layout)
    lay = np.zeros((pop_size, t.shape[0]), np.int32)
    ok = np.zeros(pop_size, np.int32)
    lib().orc_seed_trials(C.c_int32(t.shape[0]), C.c_int32(C_cap), C.c_int32(D), C.c_int32(R), C.c_int32(width),
                          C.c_uint64(seed), _p(t), _p(sl), C.c_int32(pop_size), _p(lay), _p(ok))
    return lay, ok


def edp_pair(q, layouts, R: int, D: int, width: int, seed: int, edp_of_dp=None) -> np.ndarray:
    """EDPAwarePair on every member j >= 1 of `layouts` [P][N]; returns the re-paired layouts."""
    q = _i32(q)
    lay = _i32(layouts).copy()
    Ppop, N = lay.shape
    _, L, P = q.shape
    edp = np.arange(D, dtype=np.int32) if edp_of_dp is None else _i32(edp_of_dp)
    G = int(edp.max()) + 1
    lib().orc_edp_pair(C.c_int32(N), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(G), C.c_int32(R),
                       C.c_int32(width), C.c_uint64(seed), _p(q), _p(edp), C.c_int32(Ppop), _p(lay))
    return lay


def canonicalize(layout, R: int, D: int, edp_of_dp=None) -> np.ndarray:
    lay = _i32(layout)
    edp = np.arange(D, dtype=np.int32) if edp_of_dp is None else _i32(edp_of_dp)
    out = np.zeros_like(lay)
    lib().orc_canonicalize(C.c_int32(lay.shape[0]), C.c_int32(D), C.c_int32(int(edp.max()) + 1), C.c_int32(R),
                           _p(edp), _p(lay), _p(out))
    return out


def coassign_q20(la, lb) -> int:
    la, lb = _i32(la), _i32(lb)
    return int(lib().orc_coassign_q20(C.c_int32(la.shape[0]), _p(la), _p(lb)))


def sw_sketch(lengths, q, layout, R: int, C_cap: int, D: int, top_k: int, nproj: int, seed: int, edp_of_dp=None):
    """Sorted projections [nproj][R] of the row features."""
    t, q, lay = _i32(lengths), _i32(q), _i32(layout)
    _, L, P = q.shape
    edp = np.arange(D, dtype=np.int32) if edp_of_dp is None else _i32(edp_of_dp)
    phi = np.zeros((nproj, R), np.int64)
    lib().orc_sw_sketch(C.c_int32(t.shape[0]), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(int(edp.max()) + 1),
                        C.c_int32(R), C.c_int32(C_cap), C.c_int32(top_k), C.c_int32(nproj), C.c_uint64(seed),
                        _p(t), _p(q), _p(edp), _p(lay), _p(phi))
    return phi


def select_population(lengths, q, layouts, scores, R: int, C_cap: int, D: int, top_k: int, nproj: int, eta_q16: int,
                      seed: int, edp_of_dp=None, want_dist: bool = False):
    """CanonicalMap + QualityDiversitySelect: returns dict(layouts, n_distinct, order[, dist])."""
    t, q = _i32(lengths), _i32(q)
    lay = _i32(layouts).copy()
    sc = np.ascontiguousarray(scores, dtype=np.int64)
    Ppop, N = lay.shape
    _, L, P = q.shape
    edp = np.arange(D, dtype=np.int32) if edp_of_dp is None else _i32(edp_of_dp)
    nd = C.c_int32(0)
    order = np.zeros(Ppop, np.int32)
    dist = np.zeros((Ppop, Ppop), np.int64) if want_dist else None
    lib().orc_select_population(C.c_int32(N), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(int(edp.max()) + 1),
                                C.c_int32(R), C.c_int32(C_cap), C.c_int32(top_k), C.c_int32(nproj), C.c_int64(eta_q16),
                                C.c_uint64(seed), _p(t), _p(q), _p(edp), C.c_int32(Ppop), _p(sc), _p(lay),
                                C.byref(nd), _p(order), _p(dist))
    out = dict(layouts=lay, n_distinct=int(nd.value), order=order)
    if want_dist:
        out["dist"] = dist
    return out


# ---- scoring ----------------------------------------------------------------------------
def _edp(D: int, edp_of_dp) -> np.ndarray:
    return np.arange(D, dtype=np.int32) if edp_of_dp is None else _i32(edp_of_dp)


def eval_layouts(lengths, q, layouts, R: int, C_cap: int, D: int, edp_of_dp=None,
                 alpha=(1.0, 1.0), beta=(0.0, 1.0)) -> Dict[str, np.ndarray]:
    t = _i32(lengths)
    q = _i32(q)
    lay = _i32(layouts)
    if lay.ndim == 1:
        lay = lay[None, :]
    n, N = lay.shape
    _, L, P = q.shape
    edp = _edp(D, edp_of_dp)
    G = int(edp.max()) + 1
    al, be = _f64(alpha), _f64(beta)
    K = R * D
    out = dict(T=np.zeros((n, K), np.int64), Q=np.zeros((n, K), np.int64), cnt=np.zeros((n, K), np.int32),
               W=np.zeros((n, R, G, L, P), np.int32), Afx=np.zeros((n, R, G), np.int64),
               Efx=np.zeros((n, R, G), np.int64), U=np.zeros((n, G), np.int64),
               score=np.zeros((n, 3), np.int64))
    lib().orc_eval(C.c_int32(N), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(G), C.c_int32(R),
                   C.c_int32(C_cap), _p(edp), C.c_int32(al.shape[0]), _p(al), _p(be), _p(t), _p(q),
                   C.c_int32(n), _p(lay), _p(out["T"]), _p(out["Q"]), _p(out["cnt"]), _p(out["W"]),
                   _p(out["Afx"]), _p(out["Efx"]), _p(out["U"]), _p(out["score"]))
    return out


def eval_f64(lengths, q, layout, R: int, C_cap: int, D: int, edp_of_dp=None,
             alpha=(1.0, 1.0), beta=(0.0, 1.0)) -> np.ndarray:
    t = _i32(lengths)
    q = _i32(q)
    lay = _i32(layout)
    _, L, P = q.shape
    edp = _edp(D, edp_of_dp)
    G = int(edp.max()) + 1
    al, be = _f64(alpha), _f64(beta)
    out = np.zeros(3, np.float64)
    lib().orc_eval_f64(C.c_int32(t.shape[0]), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(G),
                       C.c_int32(R), C.c_int32(C_cap), _p(edp), C.c_int32(al.shape[0]), _p(al), _p(be),
                       _p(t), _p(q), _p(lay), _p(out))
    return out


def diagnostics(lengths, q, Lagg, pi, layout, R: int, C_cap: int, D: int, edp_of_dp=None,
                alpha=(1.0, 1.0), beta=(0.0, 1.0)) -> Dict[str, float]:
    """CV_global before/after placement, S_EP, T_EP, eta_EP, attention and joint proxies of a layout."""
    t = _i32(lengths)
    q = _i32(q)
    Lagg = np.ascontiguousarray(Lagg, np.int64)
    pi = _i32(pi)
    lay = _i32(layout)
    _, L, P = q.shape
    E = Lagg.shape[1]
    edp = _edp(D, edp_of_dp)
    G = int(edp.max()) + 1
    al, be = _f64(alpha), _f64(beta)
    cv = np.zeros(2)
    peaks = np.zeros(3, np.int64)
    aj = np.zeros(2)
    eta = C.c_double(0.0)
    lib().orc_diagnostics(C.c_int32(t.shape[0]), C.c_int32(L), C.c_int32(E), C.c_int32(P), C.c_int32(D), C.c_int32(G),
                          C.c_int32(R), C.c_int32(C_cap), _p(edp), C.c_int32(al.shape[0]), _p(al), _p(be), _p(t), _p(q),
                          _p(Lagg), _p(pi), _p(lay), _p(cv), _p(peaks), _p(aj), C.byref(eta))
    return dict(cv_identity=float(cv[0]), cv_placed=float(cv[1]), s_ep=int(peaks[0]), t_ep=int(peaks[1]),
                n_ep=int(peaks[2]), eta_ep=float(eta.value), attention=float(aj[0]), joint=float(aj[1]))


def score_scale(C_cap: int) -> int:
    """SC: the integer that stands for 1.0 of the paper's normalised cost."""
    return (C_cap * C_cap) << 8


# ---- annealing --------------------------------------------------------------------------
def energy(score) -> int:
    """Scalar search energy of a score tuple (Eq. pa-energy), in score units."""
    s = np.ascontiguousarray(score, np.int64)
    return int(lib().orc_energy(_p(s)))


def propose_once(lengths, q, layout, R: int, C_cap: int, D: int, A, B, rho_q32: int, guide_q32: int,
                 edp_of_dp=None, alpha=(1.0, 1.0), beta=(0.0, 1.0)):
    """One GuidedProposal draw (Section 4.1.2) on `layout` from the random words A[4], B[4].

    Returns (move, feasible) with move = dict(reloc, i, i2, c1, c2)."""
    t = _i32(lengths)
    q = _i32(q)
    lay = _i32(layout)
    _, L, P = q.shape
    edp = _edp(D, edp_of_dp)
    G = int(edp.max()) + 1
    al, be = _f64(alpha), _f64(beta)
    Aw = np.ascontiguousarray(A, np.uint32)
    Bw = np.ascontiguousarray(B, np.uint32)
    mv = np.zeros(5, np.int32)
    ok = lib().orc_propose_once(C.c_int32(t.shape[0]), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(G),
                                C.c_int32(R), C.c_int32(C_cap), _p(edp), C.c_int32(al.shape[0]), _p(al), _p(be),
                                _p(t), _p(q), _p(lay), _p(Aw), _p(Bw), C.c_uint64(rho_q32), C.c_uint64(guide_q32),
                                _p(mv))
    return dict(reloc=int(mv[0]), i=int(mv[1]), i2=int(mv[2]), c1=int(mv[3]), c2=int(mv[4])), bool(ok)


def anneal(lengths, q, init_layouts, R: int, C_cap: int, D: int, *, n_levels: int, steps: int,
           t0: float, t_ratio: float, p_reloc: float, p_guide: float, seed: int,
           edp_of_dp=None, alpha=(1.0, 1.0), beta=(0.0, 1.0), full_rescore: bool = False,
           n_threads: int = 1, trace: bool = True) -> Dict[str, np.ndarray]:
    t = _i32(lengths)
    q = _i32(q)
    init = _i32(init_layouts)
    Ppop, N = init.shape
    _, L, P = q.shape
    edp = _edp(D, edp_of_dp)
    G = int(edp.max()) + 1
    al, be = _f64(alpha), _f64(beta)
    nl = n_levels
    out = dict(best_layout=np.zeros(N, np.int32), best_score=np.zeros(3, np.int64),
               final_pop=np.zeros((Ppop, N), np.int32), counters=np.zeros(4, np.int64))
    if trace:
        out.update(term=np.zeros((nl, Ppop, 3), np.int64), best=np.zeros((nl, Ppop, 3), np.int64),
                   best_step=np.zeros((nl, Ppop), np.int32), digest=np.zeros((nl, Ppop), np.uint64),
                   anc=np.zeros((max(nl - 1, 0), Ppop), np.int32), incumbent=np.zeros((nl, 3), np.int64))
    g = out.get
    status = lib().orc_anneal(
        C.c_int32(N), C.c_int32(L), C.c_int32(P), C.c_int32(D), C.c_int32(G), C.c_int32(R),
        C.c_int32(C_cap), _p(edp), C.c_int32(al.shape[0]), _p(al), _p(be), _p(t), _p(q),
        C.c_int32(Ppop), _p(init), C.c_int32(nl), C.c_int32(steps), C.c_double(t0), C.c_double(t_ratio),
        C.c_double(p_reloc), C.c_double(p_guide), C.c_uint64(seed), C.c_int32(int(full_rescore)),
        C.c_int32(n_threads), _p(g("term")), _p(g("best")), _p(g("best_step")), _p(g("digest")),
        _p(g("anc")), _p(g("incumbent")), _p(out["counters"]), _p(out["best_layout"]),
        _p(out["best_score"]), _p(out["final_pop"]))
    out["status"] = int(status)
    return out


def plan(window, *, pop_size: Optional[int] = None, n_levels: Optional[int] = None,
         steps: Optional[int] = None, edp_of_dp=None, n_threads: int = 1,
         full_rescore: bool = False, trace: bool = True) -> Dict[str, np.ndarray]:
    """The whole hot path on one window: check, aggregate, LPT, project, R*/FFD, anneal."""
    s = window.spec
    bad = check_window(window.lengths, window.demand, s.top_k, s.token_cap)
    if bad:
        raise ValueError(f"window fails the input checks at sample {bad - 1}")
    Lagg = aggregate(window.demand)
    pi, Gload = lpt(Lagg, s.ep_width)
    q = project(window.demand, pi, s.ep_width)
    R, cert, seed_layout = pack_ffd(window.lengths, s.token_cap, s.dp_width)
    if R == 0:
        raise ValueError("no feasible row count")
    Ppop = pop_size or s.pop_size
    init = np.tile(seed_layout[None, :], (Ppop, 1))
    res = anneal(window.lengths, q, init, R, s.token_cap, s.dp_width,
                 n_levels=n_levels or s.n_levels, steps=steps or s.steps_per_level,
                 t0=s.t0, t_ratio=s.t_ratio, p_reloc=s.p_reloc, p_guide=s.p_guide, seed=s.anneal_seed,
                 edp_of_dp=edp_of_dp, alpha=s.alpha, beta=s.beta, full_rescore=full_rescore,
                 n_threads=n_threads, trace=trace)
    res.update(Lagg=Lagg, pi=pi, rank_load=Gload, q=q, n_rows=R, certified=cert, seed_layout=seed_layout)
    return res
