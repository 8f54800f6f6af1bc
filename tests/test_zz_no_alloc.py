"""The allocation-free scoring entry point against the ordinary one.

Some callers of this library cannot allocate device memory while they run: the planner may
sit inside a training or serving loop whose framework owns every free byte of the GPU, or in
a section where cudaMalloc/cudaFree would stall the device.  For them the library offers
rp_eval_layouts_noalloc, whose working memory is a fixed array inside the library image.
This file checks, through the C ABI, that it returns exactly what rp_eval_population returns
and what the CPU oracle computes for the same layouts, twice in a row (the fixed array keeps the
previous call's contents), that the second call leaves the free device memory and the
framework's pool as it found them, and that it refuses sizes beyond its fixed limits and host
pointers.  It is collected last on purpose.
"""
import numpy as np
import pytest

import oracle
import paper_2608_12146_b200.binding as rp
from paper_2608_12146_b200.windows import custom_spec, make_window

pytestmark = pytest.mark.gpu


def planned_context(w, pop=4, edp=None, min_rows=0):
    s = w.spec
    ctx = rp.rp_window_load(w.lengths, w.demand, top_k=s.top_k, token_cap=s.token_cap, dp_width=s.dp_width,
                            ep_width=s.ep_width, pop_size=pop, edp_of_dp=edp, alpha=s.alpha, beta=s.beta,
                            min_rows=min_rows)
    rp.rp_place_experts(ctx)
    rows, _ = rp.rp_pack_rows(ctx)
    return ctx, rows


@pytest.mark.parametrize("case", ["medium", "shared_shards"])
def test_noalloc_scores_equal_the_ordinary_entry_point_twice(case):
    import torch
    if case == "medium":
        w, edp, min_rows = make_window("medium"), None, 0
    else:
        w = make_window(custom_spec("noalloc", 96, 5, 16, 2, 4096, 4, 4, 8, 100, data_seed=77))
        edp, min_rows = [0, 0, 1, 1], 3
    s = w.spec
    ctx, rows = planned_context(w, edp=edp, min_rows=min_rows)
    pi, _ = oracle.lpt(oracle.aggregate(w.demand), s.ep_width)
    q = oracle.project(w.demand, pi, s.ep_width)
    rng = np.random.default_rng(3)
    for call, n in enumerate((7, 5)):          # two calls in a row, the second one smaller
        lays = rng.integers(0, rows * s.dp_width, (n, s.n_samples)).astype(np.int32)
        want_fx, want_f64 = rp.rp_eval_population(ctx, lays)
        d_lay = torch.from_numpy(lays).cuda()
        d_fx = torch.full((n, 3), -1, dtype=torch.int64, device="cuda")
        d_f64 = torch.full((n, 3), -1.0, dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        free0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
        rp.rp_eval_layouts_noalloc(ctx, d_lay, d_fx, d_f64)
        free1, reserved1 = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
        if call == 1:                          # the first call may still load the kernels' code
            assert (free1, reserved1) == (free0, reserved0)
        got_fx, got_f64 = d_fx.cpu().numpy(), d_f64.cpu().numpy()
        assert (got_fx == want_fx).all(), f"call {call}"
        np.testing.assert_allclose(got_f64, want_f64, rtol=1e-9, atol=0)
        ev = oracle.eval_layouts(w.lengths, q, lays, rows, s.token_cap, s.dp_width, edp, s.alpha, s.beta)
        assert (got_fx == ev["score"]).all(), f"call {call} against the oracle"
        for j in range(n):
            real = oracle.eval_f64(w.lengths, q, lays[j], rows, s.token_cap, s.dp_width, edp, s.alpha, s.beta)
            np.testing.assert_allclose(got_f64[j], real, rtol=1e-9, atol=0)
    rp.rp_destroy(ctx)


def test_noalloc_rejects_what_it_cannot_hold():
    import torch
    w = make_window("tiny")
    s = w.spec
    ctx, rows = planned_context(w)
    lays = np.zeros((3, s.n_samples), np.int32)
    d_fx = torch.empty((3, 3), dtype=torch.int64, device="cuda")
    with pytest.raises(rp.RpError) as e:        # host layouts would need a staging allocation
        rp.rp_eval_layouts_noalloc(ctx, lays, d_fx, None)
    assert e.value.status == -1
    big = torch.zeros((1025, s.n_samples), dtype=torch.int32, device="cuda")
    out = torch.empty((1025, 3), dtype=torch.int64, device="cuda")
    with pytest.raises(rp.RpError) as e:        # more layouts than the fixed array has counters for
        rp.rp_eval_layouts_noalloc(ctx, big, out, None)
    assert e.value.status == -5
    bad = torch.zeros((2, s.n_samples), dtype=torch.int32, device="cuda")
    bad[1, 3] = rows * s.dp_width               # a cell that does not exist
    with pytest.raises(rp.RpError) as e:
        rp.rp_eval_layouts_noalloc(ctx, bad, torch.empty((2, 3), dtype=torch.int64, device="cuda"), None)
    assert e.value.status == -1
    rp.rp_destroy(ctx)
    # the other two limits: cell ids of all layouts (n*N <= 524288) and row-shard sums (n*R*G <= 32768)
    w = make_window("large")
    s = w.spec
    ctx, rows = planned_context(w)
    for n in (300, 170):                        # 300*2048 cells; 170 layouts of R*16 row-shards each
        assert n * s.n_samples > 524288 or n * rows * s.dp_width > 32768
        lay = torch.zeros((n, s.n_samples), dtype=torch.int32, device="cuda")
        with pytest.raises(rp.RpError) as e:
            rp.rp_eval_layouts_noalloc(ctx, lay, torch.empty((n, 3), dtype=torch.int64, device="cuda"), None)
        assert e.value.status == -5
    rp.rp_destroy(ctx)
