"""Thin ctypes binding of the C-ABI library (argument marshalling only).

Function names and argument order follow ``include/routepack.h``.  Arrays may be numpy
arrays (host memory) or torch tensors (host or CUDA); outputs are allocated here when the
caller passes none.  Nothing in this module computes any step of the method: if the CUDA
library cannot be loaded, every call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_lib = None

STATUS_NAMES = {0: "RP_OK", -1: "RP_ERR_ARG", -2: "RP_ERR_SHAPE", -3: "RP_ERR_CONSERVATION",
                -4: "RP_ERR_INFEASIBLE", -5: "RP_ERR_RANGE", -6: "RP_ERR_CUDA", -7: "RP_ERR_STATE",
                -8: "RP_ERR_TIMEOUT", -9: "RP_ERR_INVALID_PLAN"}
RP_OK = 0

EXPORTS = ("rp_window_load", "rp_place_experts", "rp_pack_rows", "rp_seed_population", "rp_pair_population", "rp_select_population", "rp_init_population", "rp_eval_population", "rp_eval_layouts_noalloc", "rp_diagnostics", "rp_anneal",
           "rp_best", "rp_destroy", "rp_release_cached_memory", "rp_strerror", "rp_last_cuda_error", "rp_debug_dump",
           "rp_debug_set_trace", "rp_debug_set_knob", "rp_debug_set_stage_timing", "rp_debug_stage_times",
           "rp_debug_nl2", "rp_debug_exp2neg", "rp_debug_philox", "rp_debug_launch_count", "rp_debug_l2_read_rate",
           "rp_debug_chain_kernel")


class RpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().rp_strerror(status).decode()
        extra = f" (cudaError {lib().rp_last_cuda_error()})" if status == -6 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}: {msg}{extra}")


class rp_config(C.Structure):
    _fields_ = [("n_samples", C.c_int32), ("n_layers", C.c_int32), ("n_experts", C.c_int32),
                ("top_k", C.c_int32), ("token_cap", C.c_int32), ("dp_width", C.c_int32),
                ("ep_width", C.c_int32), ("edp_of_dp", C.c_void_p), ("n_stages", C.c_int32),
                ("alpha", C.c_void_p), ("beta", C.c_void_p), ("pop_size", C.c_int32),
                ("min_rows", C.c_int32), ("seed", C.c_uint64)]


class rp_anneal_params(C.Structure):
    _fields_ = [("n_levels", C.c_int32), ("steps_per_level", C.c_int32), ("t0", C.c_double),
                ("t_ratio", C.c_double), ("p_reloc", C.c_double), ("p_guide", C.c_double)]


class rp_anneal_stats(C.Structure):
    _fields_ = [("proposed", C.c_int64), ("feasible", C.c_int64), ("accepted", C.c_int64),
                ("improved", C.c_int64), ("ms_chains", C.c_double),
                ("move_bytes", C.c_int64), ("gather_bytes", C.c_int64), ("staging_bytes", C.c_int64),
                ("kernel_launches", C.c_int64)]


class rp_diag(C.Structure):
    _fields_ = [("cv_identity", C.c_double), ("cv_placed", C.c_double), ("s_ep", C.c_int64), ("t_ep", C.c_int64),
                ("n_ep", C.c_int64), ("eta_ep", C.c_double), ("attention", C.c_double), ("joint", C.c_double)]


def library_path() -> str:
    return _build.LIB


def lib():
    """Load the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run paper_2608_12146_b200.build.build() (needs nvcc)")
        L = C.CDLL(path)
        L.rp_strerror.restype = C.c_char_p
        L.rp_strerror.argtypes = [C.c_int]
        L.rp_last_cuda_error.restype = C.c_int
        L.rp_destroy.restype = None
        L.rp_destroy.argtypes = [C.c_void_p]
        L.rp_window_load.argtypes = [C.POINTER(C.c_void_p), C.POINTER(rp_config), C.c_void_p, C.c_void_p, C.c_void_p]
        L.rp_place_experts.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.rp_pack_rows.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.rp_seed_population.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        L.rp_pair_population.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        L.rp_select_population.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.POINTER(C.c_int32), C.c_void_p]
        L.rp_init_population.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.POINTER(C.c_int32), C.c_void_p]
        L.rp_eval_population.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.rp_eval_layouts_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.rp_diagnostics.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(rp_diag)]
        L.rp_anneal.argtypes = [C.c_void_p, C.POINTER(rp_anneal_params), C.POINTER(rp_anneal_stats)]
        L.rp_best.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.rp_debug_dump.argtypes = [C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int64]
        L.rp_debug_set_trace.argtypes = [C.c_void_p, C.c_int]
        L.rp_debug_set_knob.argtypes = [C.c_void_p, C.c_int, C.c_int64]
        L.rp_debug_set_stage_timing.argtypes = [C.c_int]
        L.rp_debug_stage_times.argtypes = [C.c_void_p, C.c_void_p]
        L.rp_debug_nl2.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.rp_debug_exp2neg.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.rp_debug_philox.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64]
        L.rp_debug_launch_count.restype = C.c_int64
        L.rp_debug_l2_read_rate.argtypes = [C.c_int64, C.c_int32, C.POINTER(C.c_double)]
        L.rp_debug_chain_kernel.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
        _lib = L
    return _lib


def _ptr(a) -> Optional[int]:
    """Address of a numpy array or torch tensor (host or device); None stays NULL."""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        if not a.flags["C_CONTIGUOUS"]:
            raise ValueError("array must be C-contiguous")
        return a.ctypes.data
    if hasattr(a, "data_ptr"):
        if not a.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return a.data_ptr()
    raise TypeError(f"unsupported array type {type(a)}")


def _check(status: int, where: str):
    if status != RP_OK:
        raise RpError(status, where)


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)           # torch.cuda.Stream


class Context:
    """Owner of one rp_ctx*; destroyed with close() or at garbage collection."""

    def __init__(self, handle: int, cfg: rp_config, keep: tuple):
        self.handle = C.c_void_p(handle)
        self.cfg = cfg
        self._keep = keep                    # input arrays adopted by the library must stay alive
        self.n_rows = 0
        self.n_shards = 0

    def close(self):
        if self.handle:
            lib().rp_destroy(self.handle)
            self.handle = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def rp_window_load(lengths, demand, *, top_k: int, token_cap: int, dp_width: int, ep_width: int,
                   pop_size: int, edp_of_dp: Optional[Sequence[int]] = None,
                   alpha: Sequence[float] = (1.0, 1.0), beta: Sequence[float] = (0.0, 1.0),
                   min_rows: int = 0, seed: int = 0, stream=None) -> Context:
    n, l, e = tuple(demand.shape)
    al = np.ascontiguousarray(alpha, dtype=np.float64)
    be = np.ascontiguousarray(beta, dtype=np.float64)
    edp = None if edp_of_dp is None else np.ascontiguousarray(edp_of_dp, dtype=np.int32)
    cfg = rp_config(n, l, e, top_k, token_cap, dp_width, ep_width, _ptr(edp), len(al), _ptr(al), _ptr(be),
                    pop_size, min_rows, seed)
    out = C.c_void_p(None)
    st = lib().rp_window_load(C.byref(out), C.byref(cfg), _ptr(lengths), _ptr(demand), _stream_handle(stream))
    _check(st, "rp_window_load")
    ctx = Context(out.value, cfg, (lengths, demand, al, be, edp))
    ctx.n_shards = dp_width if edp is None else int(edp.max()) + 1
    return ctx


def rp_place_experts(ctx: Context, pi=None, rank_load=None):
    c = ctx.cfg
    if pi is None:
        pi = np.empty((c.n_layers, c.n_experts), np.int32)
    if rank_load is None:
        rank_load = np.empty((c.n_layers, c.ep_width), np.int64)
    _check(lib().rp_place_experts(ctx.handle, _ptr(pi), _ptr(rank_load)), "rp_place_experts")
    return pi, rank_load


def rp_pack_rows(ctx: Context) -> Tuple[int, int]:
    r, cert = C.c_int32(0), C.c_int32(0)
    _check(lib().rp_pack_rows(ctx.handle, C.byref(r), C.byref(cert)), "rp_pack_rows")
    ctx.n_rows = r.value
    return r.value, cert.value


def rp_seed_population(ctx: Context, choice_width: int) -> int:
    """Randomized seeds, one trial per member; returns how many members carry their own trial."""
    own = C.c_int32(0)
    _check(lib().rp_seed_population(ctx.handle, choice_width, C.byref(own)), "rp_seed_population")
    return own.value


def rp_pair_population(ctx: Context, choice_width: int) -> int:
    """EDPAwarePair on every member but the first; returns how many layouts changed."""
    changed = C.c_int32(0)
    _check(lib().rp_pair_population(ctx.handle, choice_width, C.byref(changed)), "rp_pair_population")
    return int(changed.value)


def rp_select_population(ctx: Context, n_proj: int = 8, eta_q16: int = 1 << 16):
    """CanonicalMap + QualityDiversitySelect over the population; returns (n_distinct, order [P_pop])."""
    nd = C.c_int32(0)
    order = np.zeros(ctx.cfg.pop_size, np.int32)
    _check(lib().rp_select_population(ctx.handle, n_proj, eta_q16, C.byref(nd), _ptr(order)), "rp_select_population")
    return int(nd.value), order


def rp_init_population(ctx: Context, n_candidates: int, choice_width: int = 4, n_proj: int = 8, eta_q16: int = 1 << 16):
    """Algorithm 2 over n_candidates fixed-row candidates; returns (n_distinct, picked [P_pop])."""
    nd = C.c_int32(0)
    picked = np.zeros(ctx.cfg.pop_size, np.int32)
    _check(lib().rp_init_population(ctx.handle, n_candidates, choice_width, n_proj, eta_q16, C.byref(nd), _ptr(picked)),
           "rp_init_population")
    return int(nd.value), picked


def rp_eval_population(ctx: Context, layouts=None, score_fx=None, score_f64=None):
    n = ctx.cfg.pop_size if layouts is None else int(layouts.shape[0])
    if score_fx is None:
        score_fx = np.empty((n, 3), np.int64)
    if score_f64 is None:
        score_f64 = np.empty((n, 3), np.float64)
    _check(lib().rp_eval_population(ctx.handle, _ptr(layouts), n, _ptr(score_fx), _ptr(score_f64)),
           "rp_eval_population")
    return score_fx, score_f64


def rp_eval_layouts_noalloc(ctx: Context, layouts, score_fx, score_f64):
    """Scores of device-resident layouts into device-resident outputs without any allocation.

    For callers that may not allocate once running (all device memory already belongs to a
    framework's pool, or an allocation would stall the device).  ``layouts`` [n][N] int32 and
    the outputs [n][3] int64 / float64 must be CUDA tensors; nothing is allocated here either.
    """
    n = int(layouts.shape[0])
    _check(lib().rp_eval_layouts_noalloc(ctx.handle, _ptr(layouts), n, _ptr(score_fx), _ptr(score_f64)),
           "rp_eval_layouts_noalloc")
    return score_fx, score_f64


def rp_diagnostics(ctx: Context, layout=None) -> dict:
    """Load-balance diagnostics of a layout (None = the incumbent) as a dict."""
    d = rp_diag()
    _check(lib().rp_diagnostics(ctx.handle, _ptr(layout), C.byref(d)), "rp_diagnostics")
    return {name: getattr(d, name) for name, _ in rp_diag._fields_}


def rp_anneal(ctx: Context, *, n_levels: int, steps_per_level: int, t0: float, t_ratio: float,
              p_reloc: float, p_guide: float, want_stats: bool = True) -> Optional[rp_anneal_stats]:
    prm = rp_anneal_params(n_levels, steps_per_level, t0, t_ratio, p_reloc, p_guide)
    stats = rp_anneal_stats() if want_stats else None
    _check(lib().rp_anneal(ctx.handle, C.byref(prm), C.byref(stats) if want_stats else None), "rp_anneal")
    return stats


def rp_best(ctx: Context, cell_of_sample=None, score_fx=None, score_f64=None):
    if cell_of_sample is None:
        cell_of_sample = np.empty(ctx.cfg.n_samples, np.int32)
    if score_fx is None:
        score_fx = np.empty(3, np.int64)
    if score_f64 is None:
        score_f64 = np.empty(3, np.float64)
    _check(lib().rp_best(ctx.handle, _ptr(cell_of_sample), _ptr(score_fx), _ptr(score_f64)), "rp_best")
    return cell_of_sample, score_fx, score_f64


def rp_destroy(ctx: Context):
    ctx.close()


def rp_release_cached_memory():
    _check(lib().rp_release_cached_memory(), "rp_release_cached_memory")


# ---- inspection hooks -------------------------------------------------------------------
DUMP = dict(LAGG=1, Q=2, SEED_LAYOUT=3, POPULATION=4, W=5, CELL_T=6, CELL_Q=7, CELL_CNT=8, ESUM=9,
            TRACE_TERM=10, TRACE_BEST=11, TRACE_BEST_STEP=12, TRACE_DIGEST=13, TRACE_ANC=14,
            TRACE_INCUMBENT=15, EVAL_W=16, SELECT_DIST=17)


def rp_debug_set_trace(ctx: Context, on: bool = True):
    _check(lib().rp_debug_set_trace(ctx.handle, int(on)), "rp_debug_set_trace")


STAGES = ("check_reduce", "placement", "projection", "pack_rows", "seed_eval", "best_check")


def rp_debug_set_stage_timing(on: bool = True):
    _check(lib().rp_debug_set_stage_timing(int(on)), "rp_debug_set_stage_timing")


def rp_debug_stage_times(ctx: Context) -> dict:
    """Device milliseconds of the front-end stages of this context (None where a stage has not run)."""
    ms = np.zeros(6, np.float64)
    _check(lib().rp_debug_stage_times(ctx.handle, _ptr(ms)), "rp_debug_stage_times")
    return {k: (float(v) if v >= 0 else None) for k, v in zip(STAGES, ms)}


KNOB = dict(BARRIER_WORKSPACE=1, WAIT_POLLS=2, STALL_ONE_CHAIN=3, RANK_LOAD_SLICES=4, LAUNCH_PER_LEVEL=5,
            CHAIN_KERNEL=6)


def rp_debug_set_knob(ctx: Context, knob: str, value: int):
    _check(lib().rp_debug_set_knob(ctx.handle, KNOB[knob], int(value)), f"rp_debug_set_knob({knob})")


def rp_debug_dump(ctx: Context, what: str, shape, dtype, index: int = 0) -> np.ndarray:
    out = np.empty(shape, dtype)
    _check(lib().rp_debug_dump(ctx.handle, DUMP[what], index, _ptr(out), out.nbytes), f"rp_debug_dump({what})")
    return out


def rp_debug_nl2(x) -> np.ndarray:
    x = np.ascontiguousarray(x, np.uint32)
    out = np.empty(x.shape, np.uint64)
    _check(lib().rp_debug_nl2(_ptr(x), _ptr(out), x.size), "rp_debug_nl2")
    return out


def rp_debug_exp2neg(z) -> np.ndarray:
    z = np.ascontiguousarray(z, np.uint64)
    out = np.empty(z.shape, np.uint64)
    _check(lib().rp_debug_exp2neg(_ptr(z), _ptr(out), z.size), "rp_debug_exp2neg")
    return out


def rp_debug_l2_read_rate(nbytes: int = 32 << 20, reps: int = 50) -> float:
    """Measured read bandwidth (GB/s) of a buffer of `nbytes` that stays in L2."""
    out = C.c_double(0.0)
    _check(lib().rp_debug_l2_read_rate(nbytes, reps, C.byref(out)), "rp_debug_l2_read_rate")
    return float(out.value)


CHAIN_KERNELS = ("k_anneal_wpc", "k_anneal_level", "k_anneal_warp")


def rp_debug_chain_kernel(ctx: Context) -> str:
    """Name of the chain kernel rp_anneal runs for this context (after rp_pack_rows)."""
    out = C.c_int32(-1)
    _check(lib().rp_debug_chain_kernel(ctx.handle, C.byref(out)), "rp_debug_chain_kernel")
    return CHAIN_KERNELS[out.value]


def rp_debug_launch_count() -> int:
    return int(lib().rp_debug_launch_count())


def rp_debug_philox(ctr, key) -> np.ndarray:
    ctr = np.ascontiguousarray(ctr, np.uint32)
    key = np.ascontiguousarray(key, np.uint32)
    out = np.empty(ctr.shape, np.uint32)
    _check(lib().rp_debug_philox(_ptr(ctr), _ptr(key), _ptr(out), ctr.shape[0]), "rp_debug_philox")
    return out
