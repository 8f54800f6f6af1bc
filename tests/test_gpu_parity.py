"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Integers, indices, placements, layouts and the whole annealing trajectory must be bit-exact;
the reported fp64 objective must agree with the oracle's real-valued evaluation to 1e-9
relative (the tolerance the benchmark spec states).
"""
import os

import numpy as np
import pytest

import oracle
import paper_2608_12146_b200.binding as rp
from paper_2608_12146_b200.windows import custom_spec, make_window

pytestmark = pytest.mark.gpu
F64_RTOL = 1e-9


def load(w, pop=None, edp=None, min_rows=0, device_inputs=False):
    s = w.spec
    t, a = w.lengths, w.demand
    if device_inputs:
        import torch
        t, a = torch.from_numpy(t).cuda(), torch.from_numpy(a).cuda()
    ctx = rp.rp_window_load(t, a, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=pop or s.pop_size, edp_of_dp=edp,
                            alpha=s.alpha, beta=s.beta, min_rows=min_rows, seed=s.anneal_seed)
    rp.rp_debug_set_trace(ctx, True)          # the parity checks read the per-level traces
    return ctx


def oracle_front(w, edp=None, min_rows=0):
    s = w.spec
    Lagg = oracle.aggregate(w.demand)
    pi, G = oracle.lpt(Lagg, s.ep_width)
    q = oracle.project(w.demand, pi, s.ep_width)
    R, cert, seed = oracle.pack_ffd(w.lengths, s.token_cap, s.dp_width, min_rows)
    return dict(Lagg=Lagg, pi=pi, G=G, q=q, R=R, cert=cert, seed=seed)


def check_front(w, ctx, ref):
    s = w.spec
    pi, load_ = rp.rp_place_experts(ctx)
    assert (rp.rp_debug_dump(ctx, "LAGG", (s.n_layers, s.n_experts), np.int64) == ref["Lagg"]).all()
    assert (pi == ref["pi"]).all()
    assert (load_ == ref["G"]).all()
    q = rp.rp_debug_dump(ctx, "Q", (s.n_samples, s.n_layers, s.ep_width), np.int32)
    assert (q == ref["q"]).all()
    R, cert = rp.rp_pack_rows(ctx)
    assert (R, cert) == (ref["R"], ref["cert"])
    assert (rp.rp_debug_dump(ctx, "SEED_LAYOUT", (s.n_samples,), np.int32) == ref["seed"]).all()
    return R


def check_eval(w, ctx, ref, edp, n=6, seed=0):
    s = w.spec
    R, D = ref["R"], s.dp_width
    rng = np.random.default_rng(seed)
    lays = rng.integers(0, R * D, (n, s.n_samples)).astype(np.int32)
    lays[0] = ref["seed"]
    fx, f64 = rp.rp_eval_population(ctx, lays)
    ev = oracle.eval_layouts(w.lengths, ref["q"], lays, R, s.token_cap, D, edp, s.alpha, s.beta)
    assert (fx == ev["score"]).all()
    G = 1 + (max(edp) if edp is not None else D - 1)
    for j in range(n):
        Wj = rp.rp_debug_dump(ctx, "EVAL_W", (R, G, s.n_layers, s.ep_width), np.int32, index=j)
        assert (Wj == ev["W"][j]).all()
        real = oracle.eval_f64(w.lengths, ref["q"], lays[j], R, s.token_cap, D, edp, s.alpha, s.beta)
        np.testing.assert_allclose(f64[j], real, rtol=F64_RTOL, atol=0)


def check_anneal(w, ctx, ref, edp, pop, levels, steps, threads=8, t_ratio=None, check_members=3, init=None, t0=None):
    s = w.spec
    t0 = s.t0 if t0 is None else t0
    R, D = ref["R"], s.dp_width
    ratio = s.t_ratio if t_ratio is None else t_ratio
    if init is None:
        init = np.tile(ref["seed"], (pop, 1))
    want = oracle.anneal(w.lengths, ref["q"], init, R, s.token_cap, D, n_levels=levels, steps=steps, t0=t0,
                         t_ratio=ratio, p_reloc=s.p_reloc, p_guide=s.p_guide, seed=s.anneal_seed,
                         edp_of_dp=edp, alpha=s.alpha, beta=s.beta, n_threads=threads)
    assert want["status"] == 0
    stats = rp.rp_anneal(ctx, n_levels=levels, steps_per_level=steps, t0=t0, t_ratio=ratio,
                         p_reloc=s.p_reloc, p_guide=s.p_guide)
    got_counters = [stats.proposed, stats.feasible, stats.accepted, stats.improved]
    assert got_counters == want["counters"].tolist()
    # the whole trajectory, level by level
    assert (rp.rp_debug_dump(ctx, "TRACE_DIGEST", (levels, pop), np.uint64) == want["digest"]).all()
    assert (rp.rp_debug_dump(ctx, "TRACE_TERM", (levels, pop, 3), np.int64) == want["term"]).all()
    assert (rp.rp_debug_dump(ctx, "TRACE_BEST", (levels, pop, 3), np.int64) == want["best"]).all()
    assert (rp.rp_debug_dump(ctx, "TRACE_BEST_STEP", (levels, pop), np.int32) == want["best_step"]).all()
    if levels > 1:
        assert (rp.rp_debug_dump(ctx, "TRACE_ANC", (levels - 1, pop), np.int32) == want["anc"]).all()
    assert (rp.rp_debug_dump(ctx, "TRACE_INCUMBENT", (levels, 3), np.int64) == want["incumbent"]).all()
    # final population and the incumbent
    popl = rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32)
    assert (popl == want["final_pop"]).all()
    layout, fx, f64 = rp.rp_best(ctx)
    assert (layout == want["best_layout"]).all() and (fx == want["best_score"]).all()
    real = oracle.eval_f64(w.lengths, ref["q"], layout, R, s.token_cap, D, edp, s.alpha, s.beta)
    np.testing.assert_allclose(f64, real, rtol=F64_RTOL, atol=0)
    # incrementally maintained state of a few members equals the oracle's full evaluation
    G = 1 + (max(edp) if edp is not None else D - 1)
    for j in sorted(set([0, pop // 2, pop - 1]))[:check_members]:
        ev = oracle.eval_layouts(w.lengths, ref["q"], popl[j], R, s.token_cap, D, edp, s.alpha, s.beta)
        assert (rp.rp_debug_dump(ctx, "W", (R, G, s.n_layers, s.ep_width), np.int32, index=j) == ev["W"][0]).all()
        assert (rp.rp_debug_dump(ctx, "CELL_T", (R * D,), np.int64, index=j) == ev["T"][0]).all()
        assert (rp.rp_debug_dump(ctx, "CELL_Q", (R * D,), np.int64, index=j) == ev["Q"][0]).all()
        assert (rp.rp_debug_dump(ctx, "CELL_CNT", (R * D,), np.int32, index=j) == ev["cnt"][0]).all()
        assert (rp.rp_debug_dump(ctx, "ESUM", (R, G), np.int64, index=j) * (256 * s.token_cap) == ev["Efx"][0]).all()
    # scoring the current population from scratch agrees with the last terminal scores
    fx_pop, _ = rp.rp_eval_population(ctx)
    assert (fx_pop == want["term"][-1]).all()
    # load-balance diagnostics of the incumbent and of the seed
    pi = oracle.lpt(ref["Lagg"], s.ep_width)[0]
    for lay, arg in ((want["best_layout"], None), (ref["seed"], ref["seed"])):
        d_want = oracle.diagnostics(w.lengths, ref["q"], ref["Lagg"], pi, lay, R, s.token_cap, D, edp, s.alpha, s.beta)
        d_got = rp.rp_diagnostics(ctx, arg)
        for key in ("s_ep", "t_ep", "n_ep"):
            assert d_got[key] == d_want[key], key
        for key in ("cv_identity", "cv_placed", "eta_ep", "attention", "joint"):
            assert abs(d_got[key] - d_want[key]) <= F64_RTOL * abs(d_want[key]), key
    return want, stats


# ---------------------------------------------------------------------------------------------
def test_device_integer_functions_bit_exact():
    rng = np.random.default_rng(0)
    ctr = rng.integers(0, 2 ** 32, (4096, 4), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0
    ctr[1] = 0xFFFFFFFF
    key = np.array([0xA4093822, 0x299F31D0], np.uint32)
    got = rp.rp_debug_philox(ctr, key)
    for i in list(range(64)) + [4095]:
        assert (got[i] == oracle.philox4x32_10(ctr[i], key)).all()
    x = np.concatenate([rng.integers(0, 2 ** 32, 20000, dtype=np.uint64).astype(np.uint32),
                        np.array([0, 1, 2, 3, 2 ** 31 - 1, 2 ** 31, 2 ** 32 - 2, 2 ** 32 - 1], np.uint32),
                        (2 ** np.arange(1, 32, dtype=np.uint64) - 1).astype(np.uint32)])
    got = rp.rp_debug_nl2(x)
    assert got.tolist() == [oracle.nl2(int(v)) for v in x]
    z = np.concatenate([rng.integers(0, 34 << 32, 20000, dtype=np.uint64),
                        np.array([0, 1, 255, 256, 2 ** 32 - 1, 2 ** 32, 32 << 32, (32 << 32) - 1, 2 ** 40, 2 ** 63], np.uint64)])
    got = rp.rp_debug_exp2neg(z)
    assert got.tolist() == [oracle.exp2neg(int(v)) for v in z]


def test_philox_against_the_curand_header(tmp_path):
    """A third implementation: cuRAND's device function, compiled here with nvcc (skipped when the
    toolkit is not on the machine), against the library's and the oracle's words."""
    import ctypes
    import shutil
    import subprocess
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not available")
    src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "aux", "philox_curand.cu")
    so = str(tmp_path / "philox_curand.so")
    res = subprocess.run([nvcc, "-O2", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler", "-fPIC", "-shared",
                          "-o", so, src], capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    lib = ctypes.CDLL(so)
    rng = np.random.default_rng(12)
    ctr = rng.integers(0, 2 ** 32, (512, 4), dtype=np.uint64).astype(np.uint32)
    ctr[0] = 0
    ctr[1] = 0xFFFFFFFF
    key = np.array([0x243F6A88, 0x85A308D3], np.uint32)
    out = np.zeros_like(ctr)
    assert lib.curand_philox_host(ctr.ctypes.data_as(ctypes.c_void_p), ctypes.c_uint32(int(key[0])), ctypes.c_uint32(int(key[1])),
                                  out.ctypes.data_as(ctypes.c_void_p), ctypes.c_int(len(ctr))) == 0
    assert (rp.rp_debug_philox(ctr, key) == out).all()
    for i in range(32):
        assert (out[i] == oracle.philox4x32_10(ctr[i], key)).all()


@pytest.mark.parametrize("per_level", [2, 1], ids=["one_launch", "launch_per_level"])
@pytest.mark.parametrize("name", ["tiny", "medium"])
def test_named_window_full_budget(name, per_level):
    """The two windows the oracle finishes in seconds, at their full population and sweeps: all
    levels in one launch (every chain is resident at once), and one launch per level."""
    w = make_window(name)
    s = w.spec
    ref = oracle_front(w)
    ctx = load(w, device_inputs=(name == "medium"))
    rp.rp_debug_set_knob(ctx, "LAUNCH_PER_LEVEL", per_level)
    check_front(w, ctx, ref)
    check_eval(w, ctx, ref, None)
    check_anneal(w, ctx, ref, None, s.pop_size, s.n_levels, s.steps_per_level)
    rp.rp_destroy(ctx)


EDGE_SPECS = [
    # name, N, L, E, k, C, D, P, edp, min_rows   (ragged sizes, non-power-of-two ranks, shared shards)
    ("ragged", 77, 3, 12, 2, 3000, 3, 3, None, 4),
    ("shared_shards", 96, 5, 16, 2, 4096, 4, 4, [0, 0, 1, 1], 3),
    ("one_shard", 64, 2, 8, 1, 2048, 4, 8, [0, 0, 0, 0], 3),
    ("interleaved", 120, 7, 24, 3, 4096, 6, 6, [0, 1, 2, 0, 1, 2], 2),
    ("one_rank", 50, 4, 5, 2, 2048, 2, 1, None, 4),
    ("wide_ranks", 90, 2, 96, 2, 4096, 2, 48, None, 5),
    ("single_slot", 40, 3, 8, 2, 2048, 1, 4, None, 6),
    ("vector_tail", 130, 9, 40, 2, 8192, 5, 20, [0, 1, 1, 2, 2], 3),
    # L*k*C*(cells per row-shard) >= 2^31: the sums over layers of the busiest ranks need 64 bits
    ("wide_sums", 72, 64, 16, 8, 1 << 20, 4, 4, [0, 0, 0, 0], 3),
    # more ranks than the register-resident placement holds (128): its shared-memory form
    ("many_ranks", 60, 2, 160, 2, 4096, 2, 160, None, 4),
]


@pytest.mark.parametrize("spec", EDGE_SPECS, ids=[e[0] for e in EDGE_SPECS])
def test_edge_shapes(spec):
    name, N, L, E, k, C, D, P, edp, min_rows = spec
    w = make_window(custom_spec(name, N, L, E, k, C, D, P, 24, 400, data_seed=len(name) * 7 + N))
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=24, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    check_eval(w, ctx, ref, edp)
    want, stats = check_anneal(w, ctx, ref, edp, 24, 8, 50, t_ratio=0.6)
    assert stats.accepted > 50
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("per_level", [2, 1], ids=["one_launch", "launch_per_level"])
def test_resampling_under_selection_pressure_small_population(per_level):
    """A cold schedule on a window whose samples really differ: resampling replaces many members
    every level, so chains adopt other members' states (and others keep theirs on chip when all
    levels run in one launch); several rp_anneal calls in a row continue from one another."""
    w = make_window(custom_spec("pressure", 140, 6, 32, 2, 4096, 4, 8, 100, 400, data_seed=321))
    s = w.spec
    edp = [0, 1, 1, 0]
    ref = oracle_front(w, edp, 3)
    ctx = load(w, pop=100, edp=edp, min_rows=3)
    rp.rp_debug_set_knob(ctx, "LAUNCH_PER_LEVEL", per_level)
    check_front(w, ctx, ref)
    want, stats = check_anneal(w, ctx, ref, edp, 100, 12, 300, t_ratio=0.5, t0=2e-5, check_members=3)    # 300 steps: two batches of step records
    anc = want["anc"]
    assert any(len(set(a.tolist())) < 60 for a in anc) and stats.gather_bytes > 0
    again = oracle.anneal(w.lengths, ref["q"], want["final_pop"], ref["R"], s.token_cap, s.dp_width, n_levels=5,
                          steps=33, t0=1e-5, t_ratio=0.7, p_reloc=0.4, p_guide=0.8, seed=s.anneal_seed,
                          edp_of_dp=edp, alpha=s.alpha, beta=s.beta)
    rp.rp_anneal(ctx, n_levels=5, steps_per_level=33, t0=1e-5, t_ratio=0.7, p_reloc=0.4, p_guide=0.8)
    assert (rp.rp_debug_dump(ctx, "TRACE_TERM", (5, 100, 3), np.int64) == again["term"]).all()
    assert (rp.rp_debug_dump(ctx, "TRACE_ANC", (4, 100), np.int32) == again["anc"]).all()
    assert (rp.rp_debug_dump(ctx, "POPULATION", (100, s.n_samples), np.int32) == again["final_pop"]).all()
    layout, fx, _ = rp.rp_best(ctx)
    best = min((tuple(want["best_score"]), 0), (tuple(again["best_score"]), 1))
    assert tuple(fx) == best[0]
    assert (layout == (want, again)[best[1]]["best_layout"]).all()
    G = 2
    for j in (0, 57, 99):
        ev = oracle.eval_layouts(w.lengths, ref["q"], again["final_pop"][j], ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)
        assert (rp.rp_debug_dump(ctx, "W", (ref["R"], G, s.n_layers, s.ep_width), np.int32, index=j) == ev["W"][0]).all()
    rp.rp_destroy(ctx)


def test_three_attention_stages_and_resume():
    """Three stage types with fractional coefficients; a second rp_anneal call continues from
    the population the first one left (the oracle is restarted from that population)."""
    w = make_window(custom_spec("stages", 100, 4, 16, 2, 4096, 4, 4, 16, 300, data_seed=99,
                                alpha=(0.5, 2.25, 1.0), beta=(0.0, 0.75, 3.0)))
    s = w.spec
    edp = [0, 0, 1, 1]
    ref = oracle_front(w, edp, 3)
    ctx = load(w, pop=16, edp=edp, min_rows=3)
    check_front(w, ctx, ref)
    check_eval(w, ctx, ref, edp)
    want, _ = check_anneal(w, ctx, ref, edp, 16, 5, 40, t_ratio=0.5)
    # resume
    again = oracle.anneal(w.lengths, ref["q"], want["final_pop"], ref["R"], s.token_cap, s.dp_width, n_levels=3,
                          steps=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3, seed=s.anneal_seed,
                          edp_of_dp=edp, alpha=s.alpha, beta=s.beta)
    rp.rp_anneal(ctx, n_levels=3, steps_per_level=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3)
    assert (rp.rp_debug_dump(ctx, "TRACE_TERM", (3, 16, 3), np.int64) == again["term"]).all()
    assert (rp.rp_debug_dump(ctx, "POPULATION", (16, s.n_samples), np.int32) == again["final_pop"]).all()
    _, fx, _ = rp.rp_best(ctx)
    assert tuple(fx) == min(tuple(want["best_score"]), tuple(again["best_score"]))
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("kernel", [1, 2], ids=["several_warps_per_chain", "warp_per_chain"])
@pytest.mark.parametrize("name,pop,levels,steps", [("large", 96, 3, 60), ("wide", 48, 2, 40), ("heavy", 64, 2, 80)])
def test_large_windows_full_shapes_reduced_budget(name, pop, levels, steps, kernel):
    """Full N, L, E, P, C, D of the three big windows (so the kernels run in the launch
    configuration of the full-size runs), with a population and step budget the oracle finishes
    quickly, on both chain kernels that take such windows; every trajectory is still compared bit
    for bit."""
    w = make_window(name)
    ref = oracle_front(w)
    ctx = load(w, pop=pop, device_inputs=True)
    rp.rp_debug_set_knob(ctx, "CHAIN_KERNEL", kernel)
    check_front(w, ctx, ref)
    check_eval(w, ctx, ref, None, n=2)
    check_anneal(w, ctx, ref, None, pop, levels, steps, check_members=2)
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("name,pop,levels,steps,t0", [("large", 1024, 20, 250, None), ("heavy", 8192, 2, 1000, None),
                                                      ("wide", 4096, 2, 250, 2e-5)])
def test_large_windows_full_population(name, pop, levels, steps, t0, threads=16):
    """The three big windows at the population the benchmark runs them at (large at its whole
    budget, heavy and wide for two levels of their real step count), every trace against the
    oracle: this is where the four-members-per-thread weights, the cumulative weights in global
    memory, the off-chip cell bookkeeping and the multi-wave rank-load free list run.  (Wide starts
    colder than its schedule does, so that already its first resampling replaces members.)"""
    w = make_window(name)
    assert pop == w.spec.pop_size and steps == w.spec.steps_per_level
    ref = oracle_front(w)
    ctx = load(w, pop=pop, device_inputs=True)
    check_front(w, ctx, ref)
    want, stats = check_anneal(w, ctx, ref, None, pop, levels, steps, threads=threads, check_members=2, t0=t0)
    assert stats.accepted > pop            # the levels did move
    if levels > 1:                          # resampling really replaced members and kept others
        anc = want["anc"][0]
        assert 1 < len(set(anc.tolist())) < pop
    rp.rp_destroy(ctx)


BARRIER_CASES = [
    # name, N, L, E, k, C, D, P, edp, min_rows, pop   (first two: warp-per-candidate kernel; last two: cooperative kernel, L*P > 512)
    ("ws_small", 96, 5, 16, 2, 4096, 4, 4, [0, 0, 1, 1], 3, 37),
    ("ws_pow2", 130, 9, 40, 2, 8192, 5, 20, None, 3, 64),
    ("ws_coop", 120, 20, 32, 2, 4096, 4, 32, None, 3, 40),
    ("ws_coop_shared", 150, 17, 64, 2, 4096, 4, 32, [0, 1, 1, 0], 2, 130),
]


@pytest.mark.parametrize("spec", BARRIER_CASES, ids=[e[0] for e in BARRIER_CASES])
@pytest.mark.parametrize("cap", [0, 64])
def test_level_barrier_paths_on_small_windows(spec, cap):
    """The level barrier with all of its shared memory (cap 0) and with next to none (cap 64: the
    cumulative weights, the cell bookkeeping and the incumbent's replay go through global memory,
    as they do for populations of thousands), on windows small enough for many levels; the
    cooperative kernel is reached with L*P > 512."""
    name, N, L, E, k, C, D, P, edp, min_rows, pop = spec
    w = make_window(custom_spec(name, N, L, E, k, C, D, P, pop, 400, data_seed=len(name) * 11 + N))
    ref = oracle_front(w, edp, min_rows)
    for slices in ((1, 2) if L * P > 512 else (0,)):       # cooperative kernel: rank loads as shared slices, and as cells
        ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
        rp.rp_debug_set_knob(ctx, "BARRIER_WORKSPACE", cap)
        rp.rp_debug_set_knob(ctx, "LAUNCH_PER_LEVEL", 1)    # the barrier in question is the one between launches
        rp.rp_debug_set_knob(ctx, "RANK_LOAD_SLICES", slices)
        rp.rp_debug_set_knob(ctx, "CHAIN_KERNEL", 1)        # (L*P > 512: the 128-thread kernel, not one warp per chain)
        check_front(w, ctx, ref)
        want, stats = check_anneal(w, ctx, ref, edp, pop, 10, 40, t_ratio=0.6, check_members=2)
        assert stats.accepted > 50 and stats.improved > 0
        if slices == 1:
            assert stats.gather_bytes == 0          # nothing is copied when members share slices
            # resume: the tables survive between calls
            s_ = w.spec
            again = oracle.anneal(w.lengths, ref["q"], want["final_pop"], ref["R"], s_.token_cap, s_.dp_width, n_levels=3,
                                  steps=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3, seed=s_.anneal_seed,
                                  edp_of_dp=edp, alpha=s_.alpha, beta=s_.beta)
            rp.rp_anneal(ctx, n_levels=3, steps_per_level=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3)
            assert (rp.rp_debug_dump(ctx, "TRACE_TERM", (3, pop, 3), np.int64) == again["term"]).all()
            assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s_.n_samples), np.int32) == again["final_pop"]).all()
            G = 1 + (max(edp) if edp is not None else D - 1)
            for j in (0, pop - 1):
                ev = oracle.eval_layouts(w.lengths, ref["q"], again["final_pop"][j], ref["R"], s_.token_cap, D, edp, s_.alpha, s_.beta)
                assert (rp.rp_debug_dump(ctx, "W", (ref["R"], G, L, P), np.int32, index=j) == ev["W"][0]).all()
        rp.rp_destroy(ctx)


OTHER_RANK_CASES = [
    # name, N, L, E, k, C, D, P, edp, min_rows, pop: L*P > 512 with rank counts that are not a power of two from 4 to 128
    ("ranks_48", 100, 12, 48, 2, 4096, 4, 48, None, 3, 30),
    ("ranks_2", 90, 300, 4, 2, 4096, 3, 2, [0, 1, 0], 2, 21),
    ("ranks_3", 64, 180, 6, 1, 3000, 2, 3, None, 4, 9),
]


@pytest.mark.parametrize("spec", OTHER_RANK_CASES, ids=[e[0] for e in OTHER_RANK_CASES])
def test_slice_pool_windows_with_other_rank_counts(spec):
    """Windows whose rank loads live in the slice pool but whose rank count the warp-per-chain
    kernel does not take (its layers must be whole 16-byte chunks): the 128-thread kernel runs them
    by default, with its element-wise scoring loop."""
    name, N, L, E, k, C, D, P, edp, min_rows, pop = spec
    w = make_window(custom_spec(name, N, L, E, k, C, D, P, pop, 400, data_seed=len(name) * 17 + N))
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    want, stats = check_anneal(w, ctx, ref, edp, pop, 6, 40, t_ratio=0.6, check_members=2)
    assert stats.accepted > 0 and stats.kernel_launches == 6 * 3
    rp.rp_destroy(ctx)


WARP_CHAIN_CASES = [
    # name, N, L, E, k, C, D, P, edp, min_rows, pop: windows with 512 < L*P <= 1024 for the warp-per-chain kernel
    ("wc_ragged", 120, 20, 32, 2, 4096, 4, 32, None, 3, 40),            # 160 chunks of 16 bytes: 5 per lane
    ("wc_shared", 151, 17, 64, 2, 4096, 4, 32, [0, 1, 1, 0], 2, 130),   # two DP slots per shard, odd sample count
    ("wc_p4", 140, 200, 16, 2, 4096, 4, 4, None, 3, 33),                # one lane per layer
    ("wc_p128", 100, 8, 128, 2, 4096, 3, 128, None, 2, 50),             # a whole warp per layer, L*P = 1024
    ("wc_cells", 700, 16, 64, 2, 8192, 64, 64, None, 5, 24),            # 320 cells
]


@pytest.mark.parametrize("spec", WARP_CHAIN_CASES, ids=[e[0] for e in WARP_CHAIN_CASES])
def test_warp_per_chain_kernel_on_small_windows(spec):
    """The chain kernel that full-size windows with thousands of chains use (one warp per chain),
    forced onto small windows: ragged chunk counts, one to 32 chunks per layer, fewer layers than
    lanes and more, shared shards, more than 256 cells; the level barrier as a launch of its own,
    with all of its shared memory and with next to none; a second rp_anneal call that resumes
    from the tables."""
    kernel = 2
    name, N, L, E, k, C, D, P, edp, min_rows, pop = spec
    w = make_window(custom_spec(name, N, L, E, k, C, D, P, pop, 400, data_seed=len(name) * 13 + N))
    ref = oracle_front(w, edp, min_rows)
    for cap in (0, 64):
        ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
        rp.rp_debug_set_knob(ctx, "CHAIN_KERNEL", kernel)
        rp.rp_debug_set_knob(ctx, "BARRIER_WORKSPACE", cap)
        check_front(w, ctx, ref)
        want, stats = check_anneal(w, ctx, ref, edp, pop, 8, 40, t_ratio=0.6, check_members=2)
        assert stats.accepted > 50 and stats.improved > 0
        assert stats.gather_bytes == 0 and stats.kernel_launches == 8 * 4       # bookkeeping (2), chains, barrier
        s_ = w.spec
        again = oracle.anneal(w.lengths, ref["q"], want["final_pop"], ref["R"], s_.token_cap, s_.dp_width, n_levels=3,
                              steps=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3, seed=s_.anneal_seed,
                              edp_of_dp=edp, alpha=s_.alpha, beta=s_.beta)
        rp.rp_anneal(ctx, n_levels=3, steps_per_level=30, t0=1e-4, t_ratio=0.5, p_reloc=0.5, p_guide=0.3)
        assert (rp.rp_debug_dump(ctx, "TRACE_TERM", (3, pop, 3), np.int64) == again["term"]).all()
        assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s_.n_samples), np.int32) == again["final_pop"]).all()
        G = 1 + (max(edp) if edp is not None else D - 1)
        for j in (0, pop - 1):
            ev = oracle.eval_layouts(w.lengths, ref["q"], again["final_pop"][j], ref["R"], s_.token_cap, D, edp, s_.alpha, s_.beta)
            assert (rp.rp_debug_dump(ctx, "W", (ref["R"], G, L, P), np.int32, index=j) == ev["W"][0]).all()
        rp.rp_destroy(ctx)


@pytest.mark.parametrize("spec", [BARRIER_CASES[0], BARRIER_CASES[2], WARP_CHAIN_CASES[0]],
                         ids=["warp_per_candidate", "cooperative", "warp_per_chain"])
def test_a_wait_that_runs_out_is_reported_and_the_context_survives(spec):
    """One chain waits on a barrier phase that nothing completes, with the poll limit cut to 10^4:
    the wait gives up, the kernels return, rp_anneal reports RP_ERR_TIMEOUT, the calls that make no
    sense afterwards are refused, and after rp_pack_rows the same context anneals again, bit for
    bit as the oracle does.  Nothing traps, faults or spins without a limit."""
    name, N, L, E, k, C, D, P, edp, min_rows, pop = spec
    w = make_window(custom_spec(name, N, L, E, k, C, D, P, pop, 400, data_seed=len(name) * 11 + N))
    s = w.spec
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    rp.rp_debug_set_knob(ctx, "CHAIN_KERNEL", 2 if name.startswith("wc_") else 1)
    rp.rp_debug_set_knob(ctx, "WAIT_POLLS", 10000)
    rp.rp_debug_set_knob(ctx, "STALL_ONE_CHAIN", 1)
    for _ in range(2):                      # the second call finds the arrival counter and the status words clean
        with pytest.raises(rp.RpError) as e:
            rp.rp_anneal(ctx, n_levels=4, steps_per_level=30, t0=s.t0, t_ratio=0.6, p_reloc=s.p_reloc, p_guide=s.p_guide)
        assert e.value.status == -8
        with pytest.raises(rp.RpError) as e:    # the population is gone: annealing on needs rp_pack_rows first
            rp.rp_anneal(ctx, n_levels=1, steps_per_level=5, t0=s.t0, t_ratio=0.6, p_reloc=s.p_reloc, p_guide=s.p_guide)
        assert e.value.status == -7
        assert rp.rp_pack_rows(ctx) == (ref["R"], ref["cert"])
    rp.rp_debug_set_knob(ctx, "STALL_ONE_CHAIN", 0)
    rp.rp_debug_set_knob(ctx, "WAIT_POLLS", 0)
    check_anneal(w, ctx, ref, edp, pop, 4, 30, t_ratio=0.6, check_members=1)
    rp.rp_destroy(ctx)


def test_full_size_properties_large():
    """Large at its full population and sweeps: properties that hold at any size (feasibility
    of every member, cached scores equal to a full rescoring, monotone incumbent, conserved
    rank loads), plus the oracle's evaluation of sampled members."""
    w = make_window("large")
    s = w.spec
    ref = oracle_front(w)
    ctx = load(w, device_inputs=True)
    R = check_front(w, ctx, ref)
    stats = rp.rp_anneal(ctx, n_levels=s.n_levels, steps_per_level=s.steps_per_level, t0=s.t0, t_ratio=s.t_ratio,
                         p_reloc=s.p_reloc, p_guide=s.p_guide)
    assert stats.proposed == s.pop_size * s.sweeps
    K = R * s.dp_width
    popl = rp.rp_debug_dump(ctx, "POPULATION", (s.pop_size, s.n_samples), np.int32)
    assert popl.min() >= 0 and popl.max() < K
    for j in range(0, s.pop_size, 37):
        assert (np.bincount(popl[j], minlength=K) >= 1).all()
        assert (np.bincount(popl[j], weights=w.lengths, minlength=K) <= s.token_cap).all()
    term = rp.rp_debug_dump(ctx, "TRACE_TERM", (s.n_levels, s.pop_size, 3), np.int64)
    fx_pop, _ = rp.rp_eval_population(ctx)
    assert (fx_pop == term[-1]).all()
    inc = [tuple(x) for x in rp.rp_debug_dump(ctx, "TRACE_INCUMBENT", (s.n_levels, 3), np.int64)]
    assert all(b <= a for a, b in zip(inc, inc[1:]))
    for j in (0, 511, 1023):
        ev = oracle.eval_layouts(w.lengths, ref["q"], popl[j], R, s.token_cap, s.dp_width)
        assert tuple(ev["score"][0]) == tuple(term[-1, j])
        Wj = rp.rp_debug_dump(ctx, "W", (R, s.dp_width, s.n_layers, s.ep_width), np.int32, index=j)
        assert (Wj == ev["W"][0]).all()
        assert (Wj.sum(axis=(0, 1)) == ref["G"]).all()          # aggregate invariance
    layout, fx, f64 = rp.rp_best(ctx)
    ev = oracle.eval_layouts(w.lengths, ref["q"], layout, R, s.token_cap, s.dp_width)
    assert tuple(ev["score"][0]) == tuple(fx) == inc[-1]
    seed_score = oracle.eval_layouts(w.lengths, ref["q"], ref["seed"], R, s.token_cap, s.dp_width)["score"][0]
    assert tuple(fx) <= tuple(seed_score)
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("case,width", [("medium", 4), ("shared", 8), ("ragged", 1), ("large", 3)])
def test_randomized_seed_population(case, width):
    """Algorithm 2's trial loop: every member's seed layout, which trials were dropped, the scores
    of the seeded population and the annealing that starts from it, all against the oracle."""
    edp, min_rows, pop = None, 0, 48
    if case == "medium":
        w = make_window("medium")
    elif case == "large":
        w = make_window("large")
    elif case == "shared":
        w = make_window(custom_spec("seeds_shared", 96, 5, 16, 2, 4096, 4, 4, pop, 400, data_seed=5))
        edp, min_rows = [0, 0, 1, 1], 3
    else:
        w = make_window(custom_spec("seeds_ragged", 77, 3, 12, 2, 3000, 3, 3, pop, 400, data_seed=6))
        min_rows = 4
    s = w.spec
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    lays, ok = oracle.seed_trials(w.lengths, ref["seed"], ref["R"], s.token_cap, s.dp_width, pop, width, s.anneal_seed)
    own = rp.rp_seed_population(ctx, width)
    assert own == int(ok.sum())
    assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == lays).all()
    ev = oracle.eval_layouts(w.lengths, ref["q"], lays, ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)
    fx, _ = rp.rp_eval_population(ctx)
    assert (fx == ev["score"]).all()
    best = min(range(pop), key=lambda j: (tuple(ev["score"][j]), j))
    layout, bfx, _ = rp.rp_best(ctx)
    assert (layout == lays[best]).all() and tuple(bfx) == tuple(ev["score"][best])
    check_anneal(w, ctx, ref, edp, pop, 4, 40, t_ratio=0.5, check_members=2, init=lays)
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("case,width", [("shared", 1), ("shared", 4), ("interleaved", 3), ("one_shard", 8),
                                        ("identity", 4), ("medium", 4), ("no_trials", 2)])
def test_edp_aware_pairing(case, width):
    """Algorithm 2's pairing operator on a randomized seed population: every member's re-paired
    layout, the scores, the incumbent and the annealing that starts from it, against the oracle."""
    pop, edp, min_rows = 40, None, 3
    if case == "medium":
        w = make_window("medium")
        min_rows = 0
    elif case in ("shared", "no_trials"):
        w = make_window(custom_spec("pair_shared", 96, 5, 16, 2, 4096, 4, 4, pop, 400, data_seed=15))
        edp = [0, 0, 1, 1]
    elif case == "interleaved":
        w = make_window(custom_spec("pair_inter", 120, 7, 24, 3, 4096, 6, 6, pop, 400, data_seed=16))
        edp, min_rows = [0, 1, 2, 0, 1, 2], 2
    elif case == "one_shard":
        w = make_window(custom_spec("pair_one", 64, 2, 8, 1, 2048, 4, 8, pop, 400, data_seed=17))
        edp = [0, 0, 0, 0]
    else:
        w = make_window(custom_spec("pair_ident", 77, 3, 12, 2, 3000, 3, 3, pop, 400, data_seed=18))
        min_rows = 4
    s = w.spec
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    if case == "no_trials":                 # straight on the length-only seed: the x_paired candidates
        lays = np.tile(ref["seed"], (pop, 1)).astype(np.int32)
    else:
        lays, _ = oracle.seed_trials(w.lengths, ref["seed"], ref["R"], s.token_cap, s.dp_width, pop, 4, s.anneal_seed)
        rp.rp_seed_population(ctx, 4)
    want = oracle.edp_pair(ref["q"], lays, ref["R"], s.dp_width, width, s.anneal_seed, edp)
    changed = rp.rp_pair_population(ctx, width)
    assert changed == int((want != lays).any(axis=1).sum())
    assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == want).all()
    ev = oracle.eval_layouts(w.lengths, ref["q"], want, ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)
    fx, _ = rp.rp_eval_population(ctx)
    assert (fx == ev["score"]).all()
    best = min(range(pop), key=lambda j: (tuple(ev["score"][j]), j))
    layout, bfx, _ = rp.rp_best(ctx)
    assert (layout == want[best]).all() and tuple(bfx) == tuple(ev["score"][best])
    check_anneal(w, ctx, ref, edp, pop, 3, 40, t_ratio=0.5, check_members=2, init=want)
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("case,eta", [("shared", 1 << 16), ("shared", 0), ("interleaved", 1 << 18),
                                      ("identity", 1 << 16), ("medium", 1 << 14), ("copies", 1 << 16)])
def test_canonical_map_and_quality_diversity_selection(case, eta):
    """Algorithm 2's last lines over a seeded and paired population: which members are one plan,
    the order the selection takes the distinct ones in, the plan distances, the new population,
    its scores, the incumbent and the annealing that starts from it, against the oracle."""
    pop, edp, min_rows, n_proj = 40, None, 3, 6
    if case == "medium":
        w = make_window("medium")
        min_rows = 0
    elif case in ("shared", "copies"):
        w = make_window(custom_spec("sel_shared", 96, 5, 16, 2, 4096, 4, 4, pop, 400, data_seed=25))
        edp = [0, 0, 1, 1]
    elif case == "interleaved":
        w = make_window(custom_spec("sel_inter", 120, 7, 24, 3, 4096, 6, 6, pop, 400, data_seed=26))
        edp, min_rows = [0, 1, 2, 0, 1, 2], 2
    else:
        w = make_window(custom_spec("sel_ident", 77, 3, 12, 2, 3000, 3, 3, pop, 400, data_seed=28))
        min_rows = 4
    s = w.spec
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    if case == "copies":            # no trials: every member is the length-only seed, re-paired with width 1 -> few classes
        lays = np.tile(ref["seed"], (pop, 1)).astype(np.int32)
        width = 2
    else:
        lays, _ = oracle.seed_trials(w.lengths, ref["seed"], ref["R"], s.token_cap, s.dp_width, pop, 4, s.anneal_seed)
        rp.rp_seed_population(ctx, 4)
        width = 3
    lays = oracle.edp_pair(ref["q"], lays, ref["R"], s.dp_width, width, s.anneal_seed, edp)
    rp.rp_pair_population(ctx, width)
    sc = oracle.eval_layouts(w.lengths, ref["q"], lays, ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)["score"]
    want = oracle.select_population(w.lengths, ref["q"], lays, sc, ref["R"], s.token_cap, s.dp_width, s.top_k, n_proj, eta,
                                    s.anneal_seed, edp, want_dist=True)
    nd, order = rp.rp_select_population(ctx, n_proj, eta)
    assert nd == want["n_distinct"]
    if case == "copies":
        assert nd < pop
    assert (order == want["order"]).all()
    got = rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32)
    assert (got == want["layouts"]).all()
    dist = rp.rp_debug_dump(ctx, "SELECT_DIST", (pop, pop), np.int64)
    reps = sorted(set(order[:nd].tolist()))
    assert (dist[np.ix_(reps, reps)] == want["dist"][np.ix_(reps, reps)]).all()
    ev = oracle.eval_layouts(w.lengths, ref["q"], want["layouts"], ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)
    fx, _ = rp.rp_eval_population(ctx)
    assert (fx == ev["score"]).all()
    layout, bfx, _ = rp.rp_best(ctx)
    assert (layout == want["layouts"][0]).all() and tuple(bfx) == tuple(ev["score"][0])     # the winner leads
    check_anneal(w, ctx, ref, edp, pop, 3, 40, t_ratio=0.5, check_members=2, init=want["layouts"])
    rp.rp_destroy(ctx)


def oracle_init_population(w, ref, edp, M, pop, width, n_proj, eta):
    """Algorithm 2 over M candidates, composed from the oracle's stages: x_length, x_paired, M - 2
    trials (shuffle -> best fit -> pairing), CanonicalMap + QualityDiversitySelect, cyclic fill."""
    s = w.spec
    R, D = ref["R"], s.dp_width
    lays, _ = oracle.seed_trials(w.lengths, ref["seed"], R, s.token_cap, D, M, width, s.anneal_seed)
    lays[1] = ref["seed"]                                  # candidate 1 starts as the length-only seed too
    cand = oracle.edp_pair(ref["q"], lays, R, D, width, s.anneal_seed, edp)
    score = lambda l: oracle.eval_layouts(w.lengths, ref["q"], l, R, s.token_cap, D, edp, s.alpha, s.beta)["score"]
    if not tuple(score(cand[1])[0]) < tuple(score(ref["seed"])[0]):
        cand[1] = ref["seed"]                              # x_paired = min_Score{x_length, pairing of x_length}
    sel = oracle.select_population(w.lengths, ref["q"], cand, score(cand), R, s.token_cap, D, s.top_k, n_proj, eta,
                                   s.anneal_seed, edp)
    nd = sel["n_distinct"]
    picked = np.array([sel["order"][m % nd] for m in range(pop)], np.int32)
    return nd, picked, cand[picked]


@pytest.mark.parametrize("case,M,pop", [("shared", 60, 24), ("shared", 10, 24), ("interleaved", 33, 33), ("medium", 80, 48),
                                        ("identity", 2, 5), ("copies", 40, 16), ("slices", 12, 40), ("slices_shared", 9, 30)])
def test_algorithm_2_as_one_call(case, M, pop):
    """rp_init_population against the composition of the oracle's stages: how many candidates are
    distinct, which candidate every member is, the members' layouts and scores, the incumbent, and
    the annealing that starts from them; with fewer, as many and more candidates than members."""
    edp, min_rows, width, n_proj, eta = None, 3, 3, 6, 1 << 16
    if case == "medium":
        w = make_window("medium")
        min_rows = 0
    elif case in ("shared", "copies"):
        w = make_window(custom_spec("a2_shared", 96, 5, 16, 2, 4096, 4, 4, pop, 400, data_seed=45))
        edp = [0, 0, 1, 1]
        if case == "copies":
            width = 1                                       # no randomness: few distinct candidates
    elif case == "interleaved":
        w = make_window(custom_spec("a2_inter", 120, 7, 24, 3, 4096, 6, 6, pop, 400, data_seed=46))
        edp, min_rows = [0, 1, 2, 0, 1, 2], 2
    elif case in ("slices", "slices_shared"):
        # rank loads in the slice pool, fewer candidates than members: the repeated members share
        # their original's slices until they rewrite them
        w = make_window(custom_spec("a2_slices", 120, 20, 32, 2, 4096, 4, 32, pop, 400, data_seed=47))
        edp = [0, 1, 1, 0] if case == "slices_shared" else None
    else:
        w = make_window(custom_spec("a2_ident", 77, 3, 12, 2, 3000, 3, 3, pop, 400, data_seed=48))
        min_rows = 4
    s = w.spec
    ref = oracle_front(w, edp, min_rows)
    ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
    check_front(w, ctx, ref)
    nd_want, picked_want, lays_want = oracle_init_population(w, ref, edp, M, pop, width, n_proj, eta)
    nd, picked = rp.rp_init_population(ctx, M, width, n_proj, eta)
    assert nd == nd_want and (picked == picked_want).all()
    if case == "copies":
        assert nd < M
    got = rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32)
    assert (got == lays_want).all()
    ev = oracle.eval_layouts(w.lengths, ref["q"], lays_want, ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)
    fx, _ = rp.rp_eval_population(ctx)
    assert (fx == ev["score"]).all()
    best = min(range(pop), key=lambda j: (tuple(ev["score"][j]), j))
    layout, bfx, _ = rp.rp_best(ctx)
    assert (layout == lays_want[best]).all() and tuple(bfx) == tuple(ev["score"][best])
    check_anneal(w, ctx, ref, edp, pop, 3, 40, t_ratio=0.5, check_members=2, init=lays_want)
    rp.rp_destroy(ctx)


def test_fuzz_random_small_windows():
    """Random shapes and search parameters (rank counts 1..48 including non powers of two, shared
    and interleaved shards, swap-only and relocation-only proposals, unguided and fully guided,
    one to four attention stages, hot and cold schedules): every trajectory against the oracle."""
    rng = np.random.default_rng(2024)
    for trial in range(24):
        P = int(rng.choice([1, 2, 3, 4, 6, 8, 16, 24, 32, 48]))
        H = int(rng.choice([1, 2, 3]))
        E = P * H
        L = int(rng.integers(1, 7))
        D = int(rng.choice([1, 2, 3, 4, 6]))
        N = int(rng.integers(max(12, 4 * D), 160))
        k = int(rng.choice([1, 2, 4]))
        C = int(rng.choice([512, 3000, 8192]))
        G = int(rng.integers(1, D + 1))
        edp = None if G == D else sorted(int(x) for x in np.concatenate([np.arange(G), rng.integers(0, G, D - G)]))
        if edp is not None and trial % 2:
            edp = [int(x) for x in rng.permutation(edp)]
        S = int(rng.integers(1, 5))
        alpha = tuple(float(x) for x in np.round(rng.uniform(0, 3, S) * 256) / 256)
        beta = tuple(float(x) for x in np.round(rng.uniform(0, 3, S) * 256) / 256)
        pop = int(rng.choice([1, 2, 5, 9, 33]))
        spec = custom_spec(f"fuzz{trial}", N, L, E, k, C, D, P, pop, 0, data_seed=1000 + trial, alpha=alpha, beta=beta,
                           p_reloc=float(rng.choice([0.0, 0.25, 0.6, 1.0])), p_guide=float(rng.choice([0.0, 0.5, 0.8, 1.0])),
                           t0=float(rng.choice([1e-5, 1e-3, 5e-2])), anneal_seed=int(rng.integers(0, 2 ** 62)))
        w = make_window(spec)
        min_rows = int(rng.integers(1, 4))
        ref = oracle_front(w, edp, min_rows)
        if ref["R"] == 0:
            continue
        ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
        check_front(w, ctx, ref)
        levels, steps = int(rng.integers(1, 5)), int(rng.choice([1, 7, 33, 130]))
        check_anneal(w, ctx, ref, edp, pop, levels, steps, t_ratio=float(rng.choice([0.3, 0.7, 1.0])), check_members=1)
        rp.rp_destroy(ctx)


def test_fuzz_warp_per_chain_kernel():
    """Random windows whose rank loads live in the slice pool (L*P of 600 to 2000 with 4 to 64
    ranks), random shard maps, attention stages, proposal mixes and schedules, on the
    warp-per-chain kernel: every trajectory against the oracle."""
    rng = np.random.default_rng(77)
    for trial in range(12):
        P = int(rng.choice([4, 8, 16, 32, 64]))
        L = int(rng.integers(600 // P + 1, 2000 // P + 1))
        H = int(rng.choice([1, 2]))
        E = P * H
        D = int(rng.choice([1, 2, 3, 4, 6]))
        N = int(rng.integers(max(16, 4 * D), 140))
        k = int(rng.choice([1, 2, 4]))
        C = int(rng.choice([3000, 8192]))
        G = int(rng.integers(1, D + 1))
        edp = None if G == D else [int(x) for x in rng.permutation(np.concatenate([np.arange(G), rng.integers(0, G, D - G)]))]
        S = int(rng.integers(1, 4))
        alpha = tuple(float(x) for x in np.round(rng.uniform(0, 3, S) * 256) / 256)
        beta = tuple(float(x) for x in np.round(rng.uniform(0, 3, S) * 256) / 256)
        pop = int(rng.choice([1, 3, 9, 40]))
        spec = custom_spec(f"wfuzz{trial}", N, L, E, k, C, D, P, pop, 0, data_seed=3000 + trial, alpha=alpha, beta=beta,
                           p_reloc=float(rng.choice([0.0, 0.25, 0.6, 1.0])), p_guide=float(rng.choice([0.0, 0.5, 0.8, 1.0])),
                           t0=float(rng.choice([1e-5, 1e-3, 5e-2])), anneal_seed=int(rng.integers(0, 2 ** 62)))
        w = make_window(spec)
        min_rows = int(rng.integers(1, 4))
        ref = oracle_front(w, edp, min_rows)
        if ref["R"] == 0:
            continue
        ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
        rp.rp_debug_set_knob(ctx, "CHAIN_KERNEL", 2)
        check_front(w, ctx, ref)
        levels, steps = int(rng.integers(1, 5)), int(rng.choice([1, 7, 33, 70]))
        _, stats = check_anneal(w, ctx, ref, edp, pop, levels, steps, t_ratio=float(rng.choice([0.3, 0.7, 1.0])), check_members=1)
        assert stats.kernel_launches == levels * 4
        rp.rp_destroy(ctx)


def test_windows_planned_at_once_on_separate_streams():
    """Three different windows (a warp-per-chain one with more than 32 KB of shared memory per
    chain, a second warp-per-chain one, and one whose rank loads live on chip) planned at the same
    time by three host threads, each on its own stream and context, several plans each: every
    plan equals the oracle's, so nothing process-wide (shared-memory limits of the kernels, memory
    pools, launch counters) is upset by another context."""
    import threading
    import torch
    cases = [("conc_a", 90, 40, 32, 2, 4096, 4, 32, None, 3, 37),        # L*P = 1280
             ("conc_b", 120, 20, 32, 2, 4096, 4, 32, [0, 1, 1, 0], 3, 25),
             ("conc_c", 96, 5, 16, 2, 4096, 4, 4, None, 3, 40)]
    jobs = []
    for name, N, L, E, k, C, D, P, edp, min_rows, pop in cases:
        w = make_window(custom_spec(name, N, L, E, k, C, D, P, pop, 400, data_seed=len(name) * 19 + N))
        s = w.spec
        ref = oracle_front(w, edp, min_rows)
        want = oracle.anneal(w.lengths, ref["q"], np.tile(ref["seed"], (pop, 1)), ref["R"], s.token_cap, D, n_levels=6, steps=40,
                             t0=s.t0, t_ratio=0.6, p_reloc=s.p_reloc, p_guide=s.p_guide, seed=s.anneal_seed, edp_of_dp=edp,
                             alpha=s.alpha, beta=s.beta)
        jobs.append((w, edp, min_rows, pop, want))
    errors = []

    def worker(job):
        try:
            w, edp, min_rows, pop, want = job
            s = w.spec
            stream = torch.cuda.Stream()
            for _ in range(6):
                ctx = rp.rp_window_load(w.lengths, w.demand, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                                        ep_width=s.ep_width, pop_size=pop, edp_of_dp=edp, alpha=s.alpha, beta=s.beta,
                                        min_rows=min_rows, seed=s.anneal_seed, stream=stream)
                rp.rp_place_experts(ctx)
                rp.rp_pack_rows(ctx)
                st = rp.rp_anneal(ctx, n_levels=6, steps_per_level=40, t0=s.t0, t_ratio=0.6, p_reloc=s.p_reloc, p_guide=s.p_guide)
                layout, fx, _ = rp.rp_best(ctx)
                assert [st.proposed, st.feasible, st.accepted, st.improved] == want["counters"].tolist()
                assert (layout == want["best_layout"]).all() and (fx == want["best_score"]).all()
                assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == want["final_pop"]).all()
                rp.rp_destroy(ctx)
        except Exception as e:          # reported by the main thread
            errors.append(repr(e))

    threads = [threading.Thread(target=worker, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


@pytest.mark.parametrize("name,pop", [("tiny", 8), ("medium", 256), ("medium", 100), ("large", 300)])
def test_annealing_without_the_inspection_hook(name, pop):
    """The per-level traces are an inspection hook: counters, final population, incumbent and
    scores without them must be those of the traced run (itself checked against the oracle
    elsewhere), over many levels, and again when rp_anneal continues from the population."""
    w = make_window(name)
    s = w.spec
    outs = []
    for trace in (True, False):
        ctx = load(w, pop=pop)
        rp.rp_debug_set_trace(ctx, trace)
        rp.rp_place_experts(ctx)
        rp.rp_pack_rows(ctx)
        res = []
        for levels, steps in ((12, 25), (5, 40)):
            st = rp.rp_anneal(ctx, n_levels=levels, steps_per_level=steps, t0=s.t0, t_ratio=0.7, p_reloc=s.p_reloc, p_guide=s.p_guide)
            layout, fx, _ = rp.rp_best(ctx)
            res.append(([st.proposed, st.feasible, st.accepted, st.improved], layout.copy(), fx.copy(),
                        rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32),
                        rp.rp_eval_population(ctx)[0]))
        outs.append(res)
        rp.rp_destroy(ctx)
    for a, b in zip(*outs):
        assert a[0] == b[0]
        for x, y in zip(a[1:], b[1:]):
            assert (x == y).all()


def test_repeated_front_end_calls_recompute():
    """rp_window_load already queues placement and packing; a second rp_place_experts or
    rp_pack_rows computes them again itself, and rp_best without a preceding rp_anneal validates
    on its own: same results on every route."""
    w = make_window(custom_spec("twice", 96, 5, 16, 2, 4096, 4, 4, 12, 400, data_seed=31))
    edp = [0, 0, 1, 1]
    ref = oracle_front(w, edp, 3)
    ctx = load(w, pop=12, edp=edp, min_rows=3)
    pi1, load1 = rp.rp_place_experts(ctx)
    pi2, load2 = rp.rp_place_experts(ctx)
    assert (pi1 == pi2).all() and (load1 == load2).all() and (pi1 == ref["pi"]).all()
    r1 = rp.rp_pack_rows(ctx)
    lay1, fx1, _ = rp.rp_best(ctx)                  # no rp_anneal yet: the seed, validated here
    r2 = rp.rp_pack_rows(ctx)
    lay2, fx2, _ = rp.rp_best(ctx)
    assert r1 == r2 and r1[0] == ref["R"]
    assert (lay1 == lay2).all() and (lay1 == ref["seed"]).all() and tuple(fx1) == tuple(fx2)
    check_eval(w, ctx, ref, edp)
    check_anneal(w, ctx, ref, edp, 12, 3, 40, t_ratio=0.5)
    lay3, fx3, _ = rp.rp_best(ctx)                  # handed over by rp_anneal
    lay4, fx4, _ = rp.rp_best(ctx)
    assert (lay3 == lay4).all() and tuple(fx3) == tuple(fx4)
    rp.rp_destroy(ctx)


def test_fuzz_seeding_stages():
    """Random shapes (one to six DP slots, one to all shards, 1..48 ranks, populations of 1..33,
    choice widths 1..32, one to nine projections, zero to large eta): trial loop, pairing and
    selection against the oracle, stage by stage."""
    rng = np.random.default_rng(77)
    done = 0
    for trial in range(16):
        P = int(rng.choice([1, 2, 3, 4, 8, 16, 48]))
        E = P * int(rng.choice([1, 2]))
        L = int(rng.integers(1, 6))
        D = int(rng.choice([1, 2, 3, 4, 6]))
        N = int(rng.integers(max(12, 4 * D), 140))
        k = int(rng.choice([1, 2, 4]))
        C = int(rng.choice([512, 3000, 8192]))
        G = int(rng.integers(1, D + 1))
        edp = None if G == D else [int(x) for x in rng.permutation(np.concatenate([np.arange(G), rng.integers(0, G, D - G)]))]
        pop = int(rng.choice([1, 2, 7, 20, 33]))
        spec = custom_spec(f"seedfuzz{trial}", N, L, E, k, C, D, P, pop, 0, data_seed=3000 + trial,
                           anneal_seed=int(rng.integers(0, 2 ** 62)))
        w = make_window(spec)
        s = w.spec
        min_rows = int(rng.integers(1, 4))
        ref = oracle_front(w, edp, min_rows)
        if ref["R"] == 0:
            continue
        ctx = load(w, pop=pop, edp=edp, min_rows=min_rows)
        check_front(w, ctx, ref)
        w1, w2 = int(rng.choice([1, 2, 5, 32])), int(rng.choice([1, 3, 32]))
        n_proj, eta = int(rng.integers(1, 10)), int(rng.choice([0, 1 << 12, 1 << 16, 1 << 24]))
        lays, ok = oracle.seed_trials(w.lengths, ref["seed"], ref["R"], s.token_cap, s.dp_width, pop, w1, s.anneal_seed)
        assert rp.rp_seed_population(ctx, w1) == int(ok.sum())
        assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == lays).all()
        paired = oracle.edp_pair(ref["q"], lays, ref["R"], s.dp_width, w2, s.anneal_seed, edp)
        assert rp.rp_pair_population(ctx, w2) == int((paired != lays).any(axis=1).sum())
        assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == paired).all()
        sc = oracle.eval_layouts(w.lengths, ref["q"], paired, ref["R"], s.token_cap, s.dp_width, edp, s.alpha, s.beta)["score"]
        want = oracle.select_population(w.lengths, ref["q"], paired, sc, ref["R"], s.token_cap, s.dp_width, s.top_k, n_proj, eta,
                                        s.anneal_seed, edp)
        nd, order = rp.rp_select_population(ctx, n_proj, eta)
        assert nd == want["n_distinct"] and (order == want["order"]).all()
        assert (rp.rp_debug_dump(ctx, "POPULATION", (pop, s.n_samples), np.int32) == want["layouts"]).all()
        check_anneal(w, ctx, ref, edp, pop, 2, 20, t_ratio=0.5, check_members=1, init=want["layouts"])
        rp.rp_destroy(ctx)
        done += 1
    assert done >= 10


def test_bad_inputs_are_host_side_errors():
    w = make_window("tiny")
    s = w.spec
    kw = dict(top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width, ep_width=s.ep_width, pop_size=4)
    bad = w.demand.copy()
    bad[7, 2, 3] += 1
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths, bad, **kw)
    assert e.value.status == -3
    neg = w.demand.copy()
    neg[3, 0, 0] -= 5
    neg[3, 0, 1] += 5
    if neg[3, 0, 0] < 0:
        with pytest.raises(rp.RpError) as e:
            rp.rp_window_load(w.lengths, neg, **kw)
        assert e.value.status == -3
    long_ = w.lengths.copy()
    long_[0] = s.token_cap + 1
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(long_, w.demand, **kw)
    assert e.value.status == -3
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths, w.demand, **dict(kw, ep_width=3))
    assert e.value.status == -2
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths[:1], w.demand[:1], **kw)
    assert e.value.status == -2
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths, w.demand, edp_of_dp=[0, 2], **kw)      # shard 1 unused
    assert e.value.status == -2
    # rank loads are 32-bit: k * C * (DP slots of one shard) must stay below 2^31; the cap itself below 2^24
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths, w.demand, **dict(kw, top_k=64, token_cap=1 << 24, edp_of_dp=[0, 0]))
    assert e.value.status == -5
    with pytest.raises(rp.RpError) as e:
        rp.rp_window_load(w.lengths, w.demand, **dict(kw, token_cap=(1 << 24) + 1))
    assert e.value.status == -5
    with pytest.raises(rp.RpError) as e:                                     # score range: (2^8*C*L*k + ...) * sum t >= 2^62
        rp.rp_window_load(w.lengths, w.demand, **dict(kw, token_cap=1 << 24, alpha=(1e6,), beta=(0.0,)))
    assert e.value.status == -5
    ctx = rp.rp_window_load(w.lengths, w.demand, **kw)
    with pytest.raises(rp.RpError) as e:
        rp.rp_pack_rows(ctx)                                                 # before rp_place_experts
    assert e.value.status == -7
    rp.rp_place_experts(ctx)
    with pytest.raises(rp.RpError) as e:
        rp.rp_anneal(ctx, n_levels=1, steps_per_level=1, t0=1e-3, t_ratio=0.5, p_reloc=0.2, p_guide=0.8)
    assert e.value.status == -7
    for call in (lambda: rp.rp_seed_population(ctx, 4), lambda: rp.rp_pair_population(ctx, 4),
                 lambda: rp.rp_select_population(ctx, 4, 1 << 16), lambda: rp.rp_init_population(ctx, 8)):
        with pytest.raises(rp.RpError) as e:
            call()                                                           # before rp_pack_rows
        assert e.value.status == -7
    R, _ = rp.rp_pack_rows(ctx)
    for call in (lambda: rp.rp_seed_population(ctx, 0), lambda: rp.rp_pair_population(ctx, 33),
                 lambda: rp.rp_select_population(ctx, 0, 1 << 16), lambda: rp.rp_select_population(ctx, 4, -1),
                 lambda: rp.rp_init_population(ctx, 1), lambda: rp.rp_init_population(ctx, 8, 0),
                 lambda: rp.rp_init_population(ctx, 8, 4, 65), lambda: rp.rp_init_population(ctx, 8, 4, 8, -1)):
        with pytest.raises(rp.RpError) as e:
            call()
        assert e.value.status == -1
    lay = np.zeros((1, s.n_samples), np.int32)
    lay[0, 5] = R * s.dp_width
    with pytest.raises(rp.RpError) as e:
        rp.rp_eval_population(ctx, lay)
    assert e.value.status == -1
    with pytest.raises(rp.RpError) as e:
        rp.rp_anneal(ctx, n_levels=0, steps_per_level=1, t0=1e-3, t_ratio=0.5, p_reloc=0.2, p_guide=0.8)
    assert e.value.status == -1
    rp.rp_anneal(ctx, n_levels=1, steps_per_level=4, t0=1e-3, t_ratio=0.5, p_reloc=0.2, p_guide=0.8)
    with pytest.raises(rp.RpError) as e:
        rp.rp_pair_population(ctx, 4)                                        # the seeding stages end with rp_anneal
    assert e.value.status == -7
    rp.rp_destroy(ctx)
    # infeasible: more DP slots than one-sample cells can fill at this cap is fine, but a window
    # whose samples cannot be split into non-empty cells within the cap is reported, not trapped
    t = np.full(6, 10, np.int32)
    a = np.zeros((6, 1, 2), np.int32)
    a[:, 0, 0] = 10
    ctx = rp.rp_window_load(t, a, top_k=1, token_cap=10, dp_width=4, ep_width=2, pop_size=2)
    rp.rp_place_experts(ctx)
    with pytest.raises(rp.RpError) as e:
        rp.rp_pack_rows(ctx)          # 6 samples of a full cell each need 6 cells; 4 and 8 are the only shapes
    assert e.value.status == -4
    rp.rp_destroy(ctx)


@pytest.mark.parametrize("E,P,N,L", [(128, 32, 70, 5), (256, 16, 37, 9), (384, 4, 33, 2), (1024, 8, 19, 3), (128, 1, 41, 3),
                                     (128, 8, 100, 2), (512, 32, 35, 4), (256, 32, 300, 3), (128, 64, 50, 2),
                                     (128, 32, 301, 32), (128, 4, 296, 32), (256, 16, 297, 48)])
def test_wide_expert_rows_front_end(E, P, N, L):
    """Rows of whole multiples of 128 experts take the 16-byte-load forms of the check + reduce and
    projection kernels (ragged sample counts: the last group of rows is partial; two shapes with 32 layers
    of 128 experts take the sequential-stream form of the check + reduce): aggregate demand,
    placement, rank demand and seed against the oracle, and every kind of bad input is still caught."""
    w = make_window(custom_spec(f"rows{E}", N, L, E, 4, 4096, 2, P, 6, 100, data_seed=E + N))
    s = w.spec
    ref = oracle_front(w, None, 2)
    for device_inputs in (False, True):
        ctx = load(w, pop=6, min_rows=2, device_inputs=device_inputs)
        check_front(w, ctx, ref)
        check_eval(w, ctx, ref, None, n=2)
        rp.rp_destroy(ctx)
    kw = dict(top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width, ep_width=s.ep_width, pop_size=2)
    for i, l, e in ((0, 0, 0), (N - 1, L - 1, E - 1), (N // 2, L // 2, 129 % E)):
        bad = w.demand.copy()
        bad[i, l, e] += 1                                   # row sum off by one
        with pytest.raises(rp.RpError) as err:
            rp.rp_window_load(w.lengths, bad, **kw)
        assert err.value.status == -3
        neg = w.demand.copy()                               # row sum right, one count negative
        neg[i, l, e] -= neg[i, l, e] + 3
        neg[i, l, (e + 5) % E] += w.demand[i, l, e] + 3
        with pytest.raises(rp.RpError) as err:
            rp.rp_window_load(w.lengths, neg, **kw)
        assert err.value.status == -3
        big = w.demand.copy()                               # sums right modulo 2^32, counts far out of range
        big[i, l, e] += 2 ** 30
        big[i, l, (e + 1) % E] += 2 ** 30
        big[i, l, (e + 2) % E] += 2 ** 30
        big[i, l, (e + 3) % E] += 2 ** 30
        with pytest.raises(rp.RpError) as err:
            rp.rp_window_load(w.lengths, big, **kw)
        assert err.value.status == -3
    long_ = w.lengths.copy()
    long_[N - 1] = 0
    with pytest.raises(rp.RpError) as err:
        rp.rp_window_load(long_, w.demand, **kw)
    assert err.value.status == -3


def test_smallest_window_and_empty_moves():
    """N == D, one row, one sample per cell: every proposal is infeasible (same cell, or a
    relocation that would empty a cell, or a swap over the cap) or a legal swap."""
    t = np.array([5, 9, 3, 7], np.int32)
    a = np.zeros((4, 2, 4), np.int32)
    rng = np.random.default_rng(5)
    for i in range(4):
        for l in range(2):
            a[i, l] = rng.multinomial(2 * t[i], [0.1, 0.2, 0.3, 0.4])
    pi, G = oracle.lpt(oracle.aggregate(a), 2)
    q = oracle.project(a, pi, 2)
    R, cert, seed = oracle.pack_ffd(t, 16, 4)
    assert R == 1
    ctx = rp.rp_window_load(t, a, top_k=2, token_cap=16, dp_width=4, ep_width=2, pop_size=3, seed=11)
    rp.rp_debug_set_trace(ctx, True)
    rp.rp_place_experts(ctx)
    assert rp.rp_pack_rows(ctx) == (R, cert)
    want = oracle.anneal(t, q, np.tile(seed, (3, 1)), R, 16, 4, n_levels=4, steps=30, t0=1e-2, t_ratio=0.5,
                         p_reloc=0.3, p_guide=0.8, seed=11)
    stats = rp.rp_anneal(ctx, n_levels=4, steps_per_level=30, t0=1e-2, t_ratio=0.5, p_reloc=0.3, p_guide=0.8)
    assert [stats.proposed, stats.feasible, stats.accepted, stats.improved] == want["counters"].tolist()
    assert (rp.rp_debug_dump(ctx, "TRACE_DIGEST", (4, 3), np.uint64) == want["digest"]).all()
    layout, fx, _ = rp.rp_best(ctx)
    assert (layout == want["best_layout"]).all() and (fx == want["best_score"]).all()
    rp.rp_destroy(ctx)
