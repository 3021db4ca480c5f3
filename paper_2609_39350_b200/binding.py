"""ctypes binding of libhap.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import weakref
import os
from typing import Optional

import numpy as np

from .build import LIB, LIB_CHECKED

MAX_TYPES, MAX_PP, MAX_LAYERS, NCOEF = 4, 32, 255, 21
INF = 1 << 62
COEF = dict(KPRE=0, KPOST=1, KP2P_INTRA=2, KP2P_INTER=3, KP2P_CROSS=4, SLAT=8, SBW=9, OPT=11,
            MW=13, MA=15, MX=17, MPRE=18, MPOST=19, KXD=20)
STATUS = ["HAP_OK", "HAP_E_INVALID", "HAP_E_NOMEM", "HAP_E_CUDA", "HAP_E_RANGE", "HAP_E_STATE", "HAP_E_INFEASIBLE"]
EXPORTS = ["hap_problem_create", "hap_problem_destroy", "hap_enumerate", "hap_get_pconfs", "hap_decode",
           "hap_eval_layer_costs", "hap_eval_layer_costs_f64", "hap_pipeline_dp", "hap_pipeline_dp_f64",
           "hap_search_range", "hap_search_range_f64",
           "hap_search_best", "hap_argmin", "hap_argmin_static", "hap_joint_bottleneck", "hap_count_cells", "hap_get_timings", "hap_launches_per_pass", "hap_eval_appendix_b", "hap_simulate_1f1b", "hap_release_cached_memory", "hap_self_check", "hap_problem_save", "hap_problem_load", "hap_problem_dims", "hap_status_str", "hap_last_error"]


class HapError(RuntimeError):
    def __init__(self, status: int, msg: str = ""):
        self.status = status
        self.name = STATUS[status] if 0 <= status < len(STATUS) else f"status {status}"
        super().__init__(f"{self.name}: {msg}" if msg else self.name)


class _Model(C.Structure):
    _fields_ = [*[(n, C.c_int32) for n in ("N", "S", "H", "E", "k", "n_shared", "F_dense", "F_exp", "nq", "nkv", "V", "GB")],
                ("beta", C.c_double), ("kind", C.c_void_p)]


class _Cluster(C.Structure):
    _fields_ = [("n_types", C.c_int32), ("P", C.c_void_p), ("C", C.c_void_p), ("node_size", C.c_void_p),
                ("bw_intra", C.c_void_p), ("n_nodes", C.c_int32), ("node_type", C.c_void_p), ("node_bw_inter", C.c_void_p)]


class _Profile(C.Structure):
    _fields_ = [("ntp", C.c_int32), ("ncp", C.c_int32), ("nmb", C.c_int32), ("nep", C.c_int32),
                ("tp_list", C.c_void_p), ("cp_list", C.c_void_p), ("mb_list", C.c_void_p), ("ep_list", C.c_void_p),
                ("tdf", C.c_void_p), ("tdb", C.c_void_p), ("tff", C.c_void_p), ("tfb", C.c_void_p),
                ("tpre", C.c_void_p), ("tpost", C.c_void_p), ("eta", C.c_void_p), ("croute", C.c_void_p),
                ("kappa", C.c_double), ("alpha", C.c_void_p), ("chi", C.c_double), ("rho", C.c_void_p),
                ("gamma", C.c_double), ("ovl_tp", C.c_double), ("ovl_cp", C.c_double), ("ovl_dp", C.c_double),
                ("act_coef", C.c_void_p), ("capf", C.c_double), ("copt", C.c_void_p), ("cap_eff", C.c_void_p),
                ("R", C.c_int32), ("xi_q", C.c_void_p), ("tau_q", C.c_void_p),
                ("n_fsize", C.c_int32), ("fsize", C.c_void_p), ("feff", C.c_void_p)]


class _Opts(C.Structure):
    _fields_ = [("npp", C.c_int32), ("ntpe", C.c_int32), ("pp_list", C.c_void_p), ("tpe_list", C.c_void_p),
                ("tp_max", C.c_int32), ("delta_q", C.c_int32), ("map_cap", C.c_uint64), ("n_rc", C.c_int32),
                ("rc_masks", C.c_void_p), ("prune", C.c_int32), ("flags", C.c_int32), ("eta_q", C.c_int32)]


class _Plan(C.Structure):
    _fields_ = [("index", C.c_uint64), *[(n, C.c_int32) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M")],
                ("rc_mask", C.c_uint32), ("pad", C.c_uint32), ("n", C.c_uint8 * MAX_PP), ("mask", C.c_uint8 * MAX_PP),
                ("r", C.c_uint8 * MAX_PP), ("T_iter", C.c_int64), ("bottleneck", C.c_int64), ("T_pipe", C.c_int64),
                ("T_sync", C.c_int64), ("T_opt", C.c_int64)]


class _Stats(C.Structure):
    _fields_ = [("n_pconf", C.c_uint64), ("n_candidates", C.c_uint64), ("n_evaluated", C.c_uint64),
                ("n_pruned", C.c_uint64), ("n_feasible", C.c_uint64), ("ms_layer_cost", C.c_float),
                ("ms_dp", C.c_float), ("ms_total", C.c_float)]


PCONF_DTYPE = np.dtype([(n, np.int32) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M", "EDP", "G",
                                                "itp", "icp", "ib", "iep", "mode", "reserved")]
                       + [("nmap", np.uint64), ("offset", np.uint64)])
CANDIDATE_DTYPE = np.dtype([("index", np.uint64), ("pconf", np.uint32), ("rc_mask", np.uint32), ("map_idx", np.uint64),
                            ("PP", np.uint8), ("pad", np.uint8, (7,)), ("mask", np.uint8, (MAX_PP,)),
                            ("link", np.uint8, (MAX_PP,))])

_lib = None


def load_library():
    """Loads libhap.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        # HAP_LIBRARY=checked selects the self-checking build of the same sources (libhap_checked.so)
        path = LIB_CHECKED if os.environ.get("HAP_LIBRARY") == "checked" else LIB
        if not os.path.exists(path):
            raise HapError(5, f"{path} is missing: run __graft_entry__.build() (nvcc, sm_100a) first")
        L = C.CDLL(path)
        L.hap_status_str.restype = C.c_char_p
        L.hap_last_error.restype = C.c_char_p
        L.hap_last_error.argtypes = [C.c_void_p]
        L.hap_problem_destroy.restype = None
        L.hap_problem_destroy.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _dev(t) -> C.c_void_p:
    """Device pointer of a CUDA torch tensor (or None)."""
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


class HapProblem:
    """Owner of a hap_problem* handle."""

    def __init__(self, handle: int, pb=None):
        self.h = C.c_void_p(handle)
        if pb is not None:
            self.N, self.T, self.n_rc = int(pb.N), int(pb.P.shape[0]), len(pb.rc_masks)
        else:                               # a loaded problem: ask the library
            n, t, r = C.c_int32(), C.c_int32(), C.c_int32()
            self.check(load_library().hap_problem_dims(self.h, C.byref(n), C.byref(t), C.byref(r)))
            self.N, self.T, self.n_rc = int(n.value), int(t.value), int(r.value)
        self.n_pconf = self.n_cand = None

    def check(self, status: int):
        if status != 0:
            msg = load_library().hap_last_error(self.h)
            raise HapError(status, msg.decode() if msg else "")

    def close(self):
        if self.h:
            load_library().hap_problem_destroy(self.h)
            self.h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


OPT_NO_MAPTAB = 1
OPT_REFINE = 2
OPT_EXACT = 4
OPT_UNIFORM = 8
OPT_HETERO_DISPATCH = 128
OPT_NO_TRIE = 16
OPT_NO_FUSE = 32
OPT_COUNT_SPLITS = 64


_ADDRESSES = {}          # id(problem) -> (weak reference to it, {field: (array as given, array as passed, address)})


def _address_memo(pb) -> dict:
    key = id(pb)
    hit = _ADDRESSES.get(key)
    if hit is not None and hit[0]() is pb:
        return hit[1]
    try:
        ref = weakref.ref(pb, lambda _r, key=key: _ADDRESSES.pop(key, None))
    except TypeError:                       # an object that cannot be referenced weakly: nothing is remembered
        return {}
    _ADDRESSES[key] = (ref, {})
    return _ADDRESSES[key][1]


def _field_address(memo: dict, pb, name: str, dtype, keep: list) -> int:
    """Address of field `name` of the problem as a C-contiguous array of `dtype` (converted if it is not one); the
    array that owns the memory is appended to `keep`."""
    a = getattr(pb, name)
    hit = memo.get(name)
    if hit is not None and hit[0] is a:
        keep.append(hit[1])
        return hit[2]
    c = a
    if not (type(c) is np.ndarray and c.dtype == dtype and c.flags.c_contiguous):     # (no copy in the usual case)
        c = np.ascontiguousarray(np.asarray(c, dtype=dtype))
    keep.append(c)
    memo[name] = (a, c, c.ctypes.data)
    return memo[name][2]


def hap_problem_create(pb, prune: int = 0, flags: int = 0) -> HapProblem:
    """Marshals a plain-data problem (see gen.problems.Problem) into the C descriptors."""
    L = load_library()
    keep = []

    # addresses of the problem's arrays, remembered per problem object and field for as long as the field holds the
    # same array object (looking an address up costs more than everything else here); kept beside the object, not in
    # it, so that copies of the problem start empty
    memo = _address_memo(pb)

    def arr(name, dtype):
        return _field_address(memo, pb, name, dtype, keep)

    mo = _Model()
    for n in ("N", "S", "H", "E", "k", "n_shared", "F_dense", "F_exp", "nq", "nkv", "V", "GB"):
        setattr(mo, n, int(getattr(pb, n)))
    mo.beta = float(pb.beta)
    mo.kind = arr("kind", np.uint8)
    cl = _Cluster()
    cl.n_types = int(pb.P.shape[0])
    cl.P, cl.C, cl.node_size = arr("P", np.int64), arr("C", np.int64), arr("node_size", np.int32)
    cl.bw_intra = arr("bw_intra", np.float64)
    cl.n_nodes = int(pb.node_type.shape[0])
    cl.node_type, cl.node_bw_inter = arr("node_type", np.int32), arr("node_bw_inter", np.float64)
    pf = _Profile()
    pf.ntp, pf.ncp, pf.nmb, pf.nep = len(pb.tp_list), len(pb.cp_list), len(pb.mb_list), len(pb.ep_list)
    for n in ("tp_list", "cp_list", "mb_list", "ep_list", "xi_q", "tau_q"):
        setattr(pf, n, arr(n, np.int32))
    for n in ("tdf", "tdb", "tff", "tfb", "tpre", "tpost", "eta", "croute", "alpha", "rho", "act_coef", "copt"):
        setattr(pf, n, arr(n, np.float64))
    for n in ("kappa", "chi", "gamma", "ovl_tp", "ovl_cp", "ovl_dp", "capf"):
        setattr(pf, n, float(getattr(pb, n)))
    pf.cap_eff = arr("cap_eff", np.int64)
    pf.R = len(pb.xi_q)
    fsize = np.ascontiguousarray(np.asarray(getattr(pb, "fsize", []), dtype=np.float64))
    feff = np.ascontiguousarray(np.asarray(getattr(pb, "feff", []), dtype=np.float64))
    keep += [fsize, feff]
    pf.n_fsize = int(fsize.shape[0])
    pf.fsize, pf.feff = (_ptr(fsize), _ptr(feff)) if pf.n_fsize else (None, None)
    so = _Opts()
    so.npp, so.ntpe = len(pb.pp_list), len(pb.tpe_list)
    so.pp_list, so.tpe_list = arr("pp_list", np.int32), arr("tpe_list", np.int32)
    so.tp_max, so.delta_q, so.map_cap = int(pb.tp_max), int(pb.delta_q), int(pb.map_cap)
    so.n_rc = len(pb.rc_masks)
    so.rc_masks = arr("rc_masks", np.uint32)
    so.prune = int(prune)
    so.flags = (int(flags) | (OPT_UNIFORM if int(getattr(pb, "uniform", 0)) else 0)
                | (OPT_HETERO_DISPATCH if int(getattr(pb, "het_coll", 0)) else 0))
    so.eta_q = int(getattr(pb, "eta_q", 0))
    out = C.c_void_p(0)
    st = L.hap_problem_create(C.byref(mo), C.byref(cl), C.byref(pf), C.byref(so), C.byref(out))
    if st != 0:
        raise HapError(st, "hap_problem_create")
    return HapProblem(out.value, pb)


def hap_problem_destroy(hp: HapProblem):
    hp.close()


def hap_enumerate(hp: HapProblem):
    a, b = C.c_uint64(), C.c_uint64()
    hp.check(load_library().hap_enumerate(hp.h, C.byref(a), C.byref(b)))
    hp.n_pconf, hp.n_cand = int(a.value), int(b.value)
    return hp.n_pconf, hp.n_cand


def hap_get_pconfs(hp: HapProblem) -> np.ndarray:
    out = np.zeros(hp.n_pconf, PCONF_DTYPE)
    hp.check(load_library().hap_get_pconfs(hp.h, _ptr(out), C.c_uint64(hp.n_pconf)))
    return out


def hap_decode(hp: HapProblem, first: int, count: int, stream=None) -> np.ndarray:
    import torch
    buf = torch.empty(max(count, 1) * CANDIDATE_DTYPE.itemsize, dtype=torch.uint8, device="cuda")
    hp.check(load_library().hap_decode(hp.h, C.c_uint64(first), C.c_uint64(count), _dev(buf), _stream(stream)))
    torch.cuda.current_stream().synchronize()
    return np.frombuffer(buf.cpu().numpy().tobytes(), dtype=CANDIDATE_DTYPE)[:count]


def hap_eval_layer_costs(hp: HapProblem, c2=None, coef=None, stream=None, want_c2=True, want_coef=True):
    """Returns (c2 [n_pconf][T][N][2], coef [n_pconf][T][NCOEF]) int64 CUDA tensors."""
    import torch
    if c2 is None and want_c2:
        c2 = torch.empty((hp.n_pconf, hp.T, hp.N, 2), dtype=torch.int64, device="cuda")
    if coef is None and want_coef:
        coef = torch.empty((hp.n_pconf, hp.T, NCOEF), dtype=torch.int64, device="cuda")
    hp.check(load_library().hap_eval_layer_costs(hp.h, _dev(c2), _dev(coef), _stream(stream)))
    return c2, coef


def hap_eval_layer_costs_f64(hp: HapProblem, stream=None):
    import torch
    c2 = torch.empty((hp.n_pconf, hp.T, hp.N, 2), dtype=torch.float64, device="cuda")
    coef = torch.empty((hp.n_pconf, hp.T, NCOEF), dtype=torch.float64, device="cuda")
    hp.check(load_library().hap_eval_layer_costs_f64(hp.h, _dev(c2), _dev(coef), _stream(stream)))
    return c2, coef


def hap_pipeline_dp(hp: HapProblem, first: int, count: int, *, partition=False, tables=False, stream=None, out=None):
    """Evaluates candidates [first, first+count).  Returns a dict of CUDA tensors."""
    import torch
    o = out or {}
    if "cost" not in o:
        o["cost"] = torch.empty(count, dtype=torch.int64, device="cuda")
        o["bottleneck"] = torch.empty(count, dtype=torch.int64, device="cuda")
        if partition:
            o["partition"] = torch.empty((count, MAX_PP), dtype=torch.uint8, device="cuda")
            o["recompute"] = torch.empty((count, MAX_PP), dtype=torch.uint8, device="cuda")
        if tables:
            o["dp_table"] = torch.full((count, MAX_PP + 1, hp.N + 1), -1, dtype=torch.int64, device="cuda")
            o["choice"] = torch.full((count, MAX_PP + 1, hp.N + 1), 254, dtype=torch.uint8, device="cuda")
    hp.check(load_library().hap_pipeline_dp(hp.h, C.c_uint64(first), C.c_uint64(count), _dev(o["cost"]),
                                            _dev(o["bottleneck"]), _dev(o.get("partition")), _dev(o.get("recompute")),
                                            _dev(o.get("dp_table")), _dev(o.get("choice")), _stream(stream)))
    return o


def hap_pipeline_dp_f64(hp: HapProblem, first: int, count: int, *, partition=False, stream=None):
    """fp64 mode: unrounded costs and bottlenecks (float64 CUDA tensors), optionally partitions and levels."""
    import torch
    o = {"cost": torch.empty(count, dtype=torch.float64, device="cuda"),
         "bottleneck": torch.empty(count, dtype=torch.float64, device="cuda")}
    if partition:
        o["partition"] = torch.empty((count, MAX_PP), dtype=torch.uint8, device="cuda")
        o["recompute"] = torch.empty((count, MAX_PP), dtype=torch.uint8, device="cuda")
    hp.check(load_library().hap_pipeline_dp_f64(hp.h, C.c_uint64(first), C.c_uint64(count), _dev(o["cost"]),
                                                _dev(o["bottleneck"]), _dev(o.get("partition")), _dev(o.get("recompute")),
                                                _stream(stream)))
    return o


def hap_search_range_f64(hp: HapProblem, first: int, count: int, stream=None):
    pl, t, b = _Plan(), C.c_double(), C.c_double()
    hp.check(load_library().hap_search_range_f64(hp.h, C.c_uint64(first), C.c_uint64(count), C.byref(pl), C.byref(t),
                                                 C.byref(b), _stream(stream)))
    d = _plan_dict(pl)
    d["T_iter_f64"], d["bottleneck_f64"] = float(t.value), float(b.value)
    return d


def _plan_dict(pl: _Plan) -> dict:
    PP = pl.PP
    return dict(index=int(pl.index), **{n: int(getattr(pl, n)) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M")},
                rc_mask=int(pl.rc_mask), n=[int(x) for x in pl.n[:PP]], mask=[int(x) for x in pl.mask[:PP]],
                r=[int(x) for x in pl.r[:PP]], T_iter=int(pl.T_iter), bottleneck=int(pl.bottleneck),
                T_pipe=int(pl.T_pipe), T_sync=int(pl.T_sync), T_opt=int(pl.T_opt))


def _stats_dict(st: _Stats) -> dict:
    return {n: (float(getattr(st, n)) if n.startswith("ms_") else int(getattr(st, n))) for n, _ in _Stats._fields_}


def hap_search_range(hp: HapProblem, first: int, count: int, stream=None):
    pl, st = _Plan(), _Stats()
    hp.check(load_library().hap_search_range(hp.h, C.c_uint64(first), C.c_uint64(count), C.byref(pl), C.byref(st),
                                             _stream(stream)))
    return _plan_dict(pl), _stats_dict(st)


def hap_search_best(hp: HapProblem, stream=None):
    pl, st = _Plan(), _Stats()
    hp.check(load_library().hap_search_best(hp.h, C.byref(pl), C.byref(st), _stream(stream)))
    return _plan_dict(pl), _stats_dict(st)


def hap_joint_bottleneck(hp: HapProblem, stream=None):
    """[n_pconf][n_rc] int64 CUDA tensor: minimum bottleneck over all stage-type sequences (-1: not homogeneous)."""
    import torch
    out = torch.empty((hp.n_pconf, hp.n_rc), dtype=torch.int64, device="cuda")
    hp.check(load_library().hap_joint_bottleneck(hp.h, _dev(out), _stream(stream)))
    return out


def hap_count_cells(hp: HapProblem, first: int, count: int, stream=None) -> int:
    """Finite-cost recurrence cells of candidates [first, first+count) (measurement aid)."""
    c = C.c_uint64()
    hp.check(load_library().hap_count_cells(hp.h, C.c_uint64(first), C.c_uint64(count), C.byref(c), _stream(stream)))
    return int(c.value)


ARGMIN_STATIC_MAX_COUNT = 1 << 26


def _check_cost_tensor(cost):
    import torch
    if not (cost.is_cuda and cost.dtype == torch.int64 and cost.is_contiguous() and cost.numel() > 0):
        raise HapError(1, "the cost array must be a non-empty contiguous int64 CUDA tensor")
    if cost.device.index is not None and cost.device.index != torch.cuda.current_device():
        raise HapError(1, "the cost array must live on the current CUDA device")


def hap_argmin_static(cost, out=None, stream=None, count=None):
    """(cost, index) minimum of an int64 CUDA tensor through the entry point that allocates nothing
    inside the library: no problem handle, scratch in the library image.  `out` is a 2-element int64
    CUDA tensor (made here with torch if not given; pass your own when the caller must not allocate).
    `count` defaults to cost.numel()."""
    import torch
    _check_cost_tensor(cost)
    if out is None:
        out = torch.empty(2, dtype=torch.int64, device=cost.device)
    if not (out.is_cuda and out.dtype == torch.int64 and out.is_contiguous() and out.numel() >= 2 and out.device == cost.device):
        raise HapError(1, "hap_argmin_static: out must be a contiguous int64 CUDA tensor of 2 elements on the cost tensor's device")
    n = cost.numel() if count is None else int(count)
    if n < 1 or n > cost.numel():
        raise HapError(4, f"hap_argmin_static: count {n} outside [1, {cost.numel()}] (the tensor's size)")
    st = load_library().hap_argmin_static(_dev(cost), C.c_uint64(n), _dev(out), _stream(stream))
    if st != 0:
        raise HapError(st, "hap_argmin_static: count must be in [1, 2^26] and the pointers non-null" if st in (1, 4) else "hap_argmin_static")
    return out


def hap_get_timings(hp: HapProblem):
    """(ms of the layer-cost kernel, ms of the DP kernel, recurrence cells) of the last DP/search call."""
    a, b, c = C.c_float(), C.c_float(), C.c_uint64()
    hp.check(load_library().hap_get_timings(hp.h, C.byref(a), C.byref(b), C.byref(c)))
    return float(a.value), float(b.value), int(c.value)


def hap_eval_appendix_b(hp: HapProblem, first: int, count: int, partition, recompute, *, detail=False, stream=None):
    """Appendix B's iteration latency of the plans (partition, recompute as returned by hap_pipeline_dp for the
    same range).  Returns {"t_iter": [count] int64, "detail": [count][3] (T_edge, T_middle, s_max) or None}."""
    import torch
    t = torch.empty(count, dtype=torch.int64, device="cuda")
    d = torch.empty((count, 3), dtype=torch.int64, device="cuda") if detail else None
    hp.check(load_library().hap_eval_appendix_b(hp.h, C.c_uint64(first), C.c_uint64(count), _dev(partition), _dev(recompute),
                                                _dev(t), _dev(d), _stream(stream)))
    return {"t_iter": t, "detail": d}


def hap_simulate_1f1b(hp: HapProblem, first: int, count: int, partition, recompute, *, detail=False, stream=None):
    """Iteration latency of the plans by an event simulation of the 1F1B schedule (partition, recompute as returned
    by hap_pipeline_dp for the same range).  Returns {"t_iter": [count] int64, "detail": [count][2] (simulated
    pipeline time, Eq. 4's pipeline term) or None}."""
    import torch
    t = torch.empty(count, dtype=torch.int64, device="cuda")
    d = torch.empty((count, 2), dtype=torch.int64, device="cuda") if detail else None
    hp.check(load_library().hap_simulate_1f1b(hp.h, C.c_uint64(first), C.c_uint64(count), _dev(partition), _dev(recompute),
                                              _dev(t), _dev(d), _stream(stream)))
    return {"t_iter": t, "detail": d}


def hap_problem_dims(hp: HapProblem):
    """(layers, device types, recomputation policies) of a problem."""
    return hp.N, hp.T, hp.n_rc


def hap_problem_save(hp: HapProblem) -> bytes:
    """The problem's inputs (model, cluster, tables, coefficients, search options) as one blob."""
    need = C.c_uint64()
    hp.check(load_library().hap_problem_save(hp.h, None, C.c_uint64(0), C.byref(need)))
    buf = C.create_string_buffer(int(need.value))
    hp.check(load_library().hap_problem_save(hp.h, buf, C.c_uint64(need.value), C.byref(need)))
    return buf.raw[:int(need.value)]


def hap_problem_load(blob: bytes) -> HapProblem:
    """A new problem on the current device from a blob written by hap_problem_save."""
    h = C.c_void_p()
    st = load_library().hap_problem_load(blob, C.c_uint64(len(blob)), C.byref(h))
    if st != 0:
        raise HapError(st, "hap_problem_load")
    return HapProblem(h.value)


def hap_self_check() -> int:
    """Check sites that fired since the last call (bit per site, 0: none); raises HAP_E_STATE unless the loaded
    library is the self-checking build."""
    sites = C.c_uint64()
    st = load_library().hap_self_check(C.byref(sites))
    if st != 0:
        raise HapError(st, "hap_self_check")
    return int(sites.value)


def hap_release_cached_memory() -> None:
    """Returns the device memory the library keeps from destroyed problems to the driver."""
    st = load_library().hap_release_cached_memory()
    if st != 0:
        raise HapError(st, "hap_release_cached_memory")


def hap_launches_per_pass(hp: HapProblem) -> int:
    """Kernels launched by one hap_pipeline_dp over every candidate plus one hap_argmin."""
    n = C.c_uint32()
    hp.check(load_library().hap_launches_per_pass(hp.h, C.byref(n)))
    return int(n.value)


def hap_argmin(hp: HapProblem, cost, stream=None):
    """(cost, index) minimum of an int64 CUDA tensor, lowest index on ties; returns a 2-element CUDA tensor."""
    import torch
    _check_cost_tensor(cost)
    out = torch.empty(2, dtype=torch.int64, device=cost.device)
    hp.check(load_library().hap_argmin(hp.h, _dev(cost), C.c_uint64(cost.numel()), _dev(out), _stream(stream)))
    return out
