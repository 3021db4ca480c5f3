"""ctypes front end of the C oracle (test infrastructure, see hap_oracle.h).

`Oracle(problem)` marshals a plain-data planning problem into the oracle's own C struct
and exposes the oracle's functions with numpy outputs.  Nothing here computes anything of
the method: it only moves arguments.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "libhap_oracle.so")
_SRC = [os.path.join(_DIR, "hap_oracle.c"), os.path.join(_DIR, "hap_oracle.h")]

MAX_TYPES, MAX_PP, MAX_N, NCOEF = 4, 32, 255, 21
INF = 1 << 62
COEF = dict(KPRE=0, KPOST=1, KP2P_INTRA=2, KP2P_INTER=3, KP2P_CROSS=4, SLAT=8, SBW=9, OPT=11,
            MW=13, MA=15, MX=17, MPRE=18, MPOST=19, KXD=20)


def build_oracle(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, floating-point contraction off)."""
    stale = force or not os.path.exists(_SO) or any(os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if stale:
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-std=c11", "-Wall", "-shared", "-fPIC",
               "-o", _SO, _SRC[0], "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


class _Problem(C.Structure):
    _fields_ = [
        *[(n, C.c_int32) for n in ("N", "S", "H", "E", "k", "n_shared", "F_dense", "F_exp", "nq", "nkv", "V", "GB")],
        ("beta", C.c_double), ("kind", C.c_void_p),
        ("T", C.c_int32), ("P", C.c_void_p), ("C", C.c_void_p), ("node_size", C.c_void_p),
        ("bw_intra", C.c_void_p), ("n_nodes", C.c_int32), ("node_type", C.c_void_p),
        ("node_bw_inter", C.c_void_p),
        ("ntp", C.c_int32), ("ncp", C.c_int32), ("nmb", C.c_int32), ("nep", C.c_int32),
        ("tp_list", C.c_void_p), ("cp_list", C.c_void_p), ("mb_list", C.c_void_p), ("ep_list", C.c_void_p),
        ("tdf", C.c_void_p), ("tdb", C.c_void_p), ("tff", C.c_void_p), ("tfb", C.c_void_p),
        ("tpre", C.c_void_p), ("tpost", C.c_void_p), ("eta", C.c_void_p), ("croute", C.c_void_p),
        ("kappa", C.c_double), ("alpha", C.c_void_p), ("chi", C.c_double), ("rho", C.c_void_p),
        ("gamma", C.c_double), ("ovl_tp", C.c_double), ("ovl_cp", C.c_double), ("ovl_dp", C.c_double),
        ("act_coef", C.c_void_p), ("capf", C.c_double), ("copt", C.c_void_p), ("cap_eff", C.c_void_p),
        ("R", C.c_int32), ("xi_q", C.c_void_p), ("tau_q", C.c_void_p),
        ("npp", C.c_int32), ("ntpe", C.c_int32), ("pp_list", C.c_void_p), ("tpe_list", C.c_void_p),
        ("tp_max", C.c_int32), ("delta_q", C.c_int32), ("map_cap", C.c_uint64),
        ("n_rc", C.c_int32), ("rc_masks", C.c_void_p), ("eta_q", C.c_int32), ("uniform", C.c_int32),
        ("n_fsize", C.c_int32), ("het_coll", C.c_int32), ("fsize", C.c_void_p), ("feff", C.c_void_p),
    ]


class PConf(C.Structure):
    _fields_ = [*[(n, C.c_int32) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M", "EDP", "G",
                                           "itp", "icp", "ib", "iep", "mode", "pad")],
                ("nmap", C.c_uint64), ("offset", C.c_uint64)]


class Mapping(C.Structure):
    _fields_ = [("PP", C.c_int32), ("mask", C.c_uint8 * MAX_PP), ("cls", C.c_uint8 * MAX_PP),
                ("ha", C.c_uint8 * MAX_PP), ("hb", C.c_uint8 * MAX_PP)]


class Result(C.Structure):
    _fields_ = [("T_iter", C.c_int64), ("bottleneck", C.c_int64), ("T_pipe", C.c_int64),
                ("T_sync", C.c_int64), ("T_opt", C.c_int64), ("n", C.c_uint8 * MAX_PP),
                ("r", C.c_uint8 * MAX_PP), ("c", C.c_int64 * MAX_PP)]


class ResultF(C.Structure):
    _fields_ = [("T_iter", C.c_double), ("bottleneck", C.c_double), ("T_pipe", C.c_double),
                ("T_sync", C.c_double), ("T_opt", C.c_double), ("n", C.c_uint8 * MAX_PP),
                ("r", C.c_uint8 * MAX_PP), ("c", C.c_double * MAX_PP)]


class AppBResult(C.Structure):
    _fields_ = [("T_iter", C.c_int64), ("T_edge", C.c_int64), ("T_middle", C.c_int64), ("T_sync", C.c_int64),
                ("T_opt", C.c_int64), ("s_max", C.c_int32), ("pad", C.c_int32)]


class SimResult(C.Structure):
    _fields_ = [("T_iter", C.c_int64), ("T_pipe_sim", C.c_int64), ("T_pipe_closed", C.c_int64), ("T_sync", C.c_int64),
                ("T_opt", C.c_int64)]


class Plan(C.Structure):
    _fields_ = [("index", C.c_uint64), ("pc", PConf), ("map", Mapping), ("rc_mask", C.c_uint32), ("res", Result)]


PCONF_DTYPE = np.dtype([(n, np.int32) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M", "EDP", "G",
                                                "itp", "icp", "ib", "iep", "mode", "pad")]
                       + [("nmap", np.uint64), ("offset", np.uint64)])

_lib = None


def lib():
    global _lib
    if _lib is None:
        build_oracle()
        L = C.CDLL(_SO)
        L.orc_multiset_count.restype = C.c_uint64
        L.orc_rank_multiset.restype = C.c_uint64
        L.orc_stage_cost.restype = C.c_int64
        L.orc_bruteforce.restype = C.c_int64
        L.orc_bruteforce_sum.restype = C.c_int64
        L.orc_joint_bottleneck.restype = C.c_int64
        L.orc_bruteforce_pipe.restype = C.c_int64
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def plan_to_dict(pl: Plan) -> dict:
    PP = pl.pc.PP
    return dict(
        index=int(pl.index),
        **{n: int(getattr(pl.pc, n)) for n in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M")},
        n=[int(x) for x in pl.res.n[:PP]], r=[int(x) for x in pl.res.r[:PP]],
        mask=[int(x) for x in pl.map.mask[:PP]], c=[int(x) for x in pl.res.c[:PP]],
        rc_mask=int(pl.rc_mask), T_iter=int(pl.res.T_iter), bottleneck=int(pl.res.bottleneck),
        T_pipe=int(pl.res.T_pipe), T_sync=int(pl.res.T_sync), T_opt=int(pl.res.T_opt))


class Oracle:
    def __init__(self, pb):
        self.pb = pb
        self.L = lib()
        keep = {}

        def arr(name, dtype):
            a = np.ascontiguousarray(np.asarray(getattr(pb, name), dtype=dtype))
            keep[name] = a
            return _ptr(a)

        s = _Problem()
        for n in ("N", "S", "H", "E", "k", "n_shared", "F_dense", "F_exp", "nq", "nkv", "V", "GB"):
            setattr(s, n, int(getattr(pb, n)))
        s.beta = float(pb.beta)
        s.kind = arr("kind", np.uint8)
        s.T = int(pb.P.shape[0])
        s.P = arr("P", np.int64); s.C = arr("C", np.int64); s.node_size = arr("node_size", np.int32)
        s.bw_intra = arr("bw_intra", np.float64); s.n_nodes = int(pb.node_type.shape[0])
        s.node_type = arr("node_type", np.int32); s.node_bw_inter = arr("node_bw_inter", np.float64)
        s.ntp, s.ncp, s.nmb, s.nep = (len(pb.tp_list), len(pb.cp_list), len(pb.mb_list), len(pb.ep_list))
        for n in ("tp_list", "cp_list", "mb_list", "ep_list", "pp_list", "tpe_list", "xi_q", "tau_q"):
            setattr(s, n, arr(n, np.int32))
        for n in ("tdf", "tdb", "tff", "tfb", "tpre", "tpost", "eta", "croute", "alpha", "rho", "act_coef", "copt"):
            setattr(s, n, arr(n, np.float64))
        s.cap_eff = arr("cap_eff", np.int64)
        for n in ("kappa", "chi", "gamma", "ovl_tp", "ovl_cp", "ovl_dp", "capf"):
            setattr(s, n, float(getattr(pb, n)))
        s.R = len(pb.xi_q)
        s.npp, s.ntpe = len(pb.pp_list), len(pb.tpe_list)
        s.tp_max, s.delta_q, s.map_cap = int(pb.tp_max), int(pb.delta_q), int(pb.map_cap)
        s.n_rc = len(pb.rc_masks)
        s.rc_masks = arr("rc_masks", np.uint32)
        s.eta_q = int(getattr(pb, "eta_q", 0))
        s.uniform = int(getattr(pb, "uniform", 0))
        s.het_coll = int(getattr(pb, "het_coll", 0))
        fsize = np.ascontiguousarray(np.asarray(getattr(pb, "fsize", []), dtype=np.float64))
        feff = np.ascontiguousarray(np.asarray(getattr(pb, "feff", []), dtype=np.float64))
        keep["fsize"], keep["feff"] = fsize, feff
        s.n_fsize = int(fsize.shape[0])
        s.fsize, s.feff = (_ptr(fsize), _ptr(feff)) if s.n_fsize else (None, None)
        self._keep = keep
        self.s = s
        self.N, self.T = int(pb.N), s.T
        self._enumerate()

    # ---- enumeration -----------------------------------------------------------------
    def _enumerate(self):
        npc, nc = C.c_uint64(), C.c_uint64()
        rc = self.L.orc_enumerate(C.byref(self.s), None, C.c_uint64(0), C.byref(npc), C.byref(nc))
        assert rc == 0
        self.pconfs = np.zeros(npc.value, dtype=PCONF_DTYPE)
        assert self.pconfs.dtype.itemsize == C.sizeof(PConf)
        rc = self.L.orc_enumerate(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(npc.value), C.byref(npc), C.byref(nc))
        assert rc == 0
        self.n_pconf, self.n_cand = int(npc.value), int(nc.value)

    def _pc(self, p: int):
        return C.byref(PConf.from_buffer(self.pconfs, p * self.pconfs.dtype.itemsize))

    def find_pconf(self, index: int) -> int:
        offs = self.pconfs["offset"]
        return int(np.searchsorted(offs, np.uint64(index), side="right") - 1)

    # ---- pieces ----------------------------------------------------------------------
    def layer_costs(self, p: int):
        """(c2 [T][N][2] int64, c2f same in fp64, coef [T][NCOEF] int64, coeff fp64)."""
        c2 = np.zeros((self.T, self.N, 2), np.int64); c2f = np.zeros((self.T, self.N, 2), np.float64)
        coef = np.zeros((self.T, NCOEF), np.int64); coeff = np.zeros((self.T, NCOEF), np.float64)
        self.L.orc_layer_costs(C.byref(self.s), self._pc(p), _ptr(c2), _ptr(c2f), _ptr(coef), _ptr(coeff))
        return c2, c2f, coef, coeff

    def decode(self, p: int, map_idx: int) -> Optional[Mapping]:
        mp = Mapping()
        rc = self.L.orc_decode(C.byref(self.s), self._pc(p), C.c_uint64(map_idx), C.byref(mp))
        return mp if rc == 0 else None

    def window(self, p: int, mp: Mapping):
        lo = np.zeros(MAX_PP, np.int32); hi = np.zeros(MAX_PP, np.int32)
        self.L.orc_window(C.byref(self.s), self._pc(p), C.byref(mp), _ptr(lo), _ptr(hi))
        PP = int(self.pconfs["PP"][p])
        return lo[:PP].copy(), hi[:PP].copy()

    def stage_cost(self, p, mp, rc_mask, c2, coef, i, a, b):
        r = C.c_int(-1)
        c = self.L.orc_stage_cost(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2), _ptr(coef),
                                  C.c_int(i), C.c_int(a), C.c_int(b), C.byref(r))
        return int(c), int(r.value)

    def candidate(self, p, mp, rc_mask, c2, coef, tables: bool = False):
        PP = int(self.pconfs["PP"][p])
        res = Result()
        dp = np.zeros((PP + 1, self.N + 1), np.int64) if tables else None
        ch = np.zeros((PP + 1, self.N + 1), np.uint8) if tables else None
        self.L.orc_candidate(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2), _ptr(coef),
                             C.byref(res), _ptr(dp) if tables else None, _ptr(ch) if tables else None)
        return res, dp, ch

    def appendix_b(self, p, mp, c2, coef, n, r) -> AppBResult:
        """Appendix B's iteration latency of a given plan (layers n and recomputation levels r per stage)."""
        res = AppBResult()
        na = np.zeros(MAX_PP, np.uint8); ra = np.zeros(MAX_PP, np.uint8)
        na[:len(n)] = n; ra[:len(r)] = r
        self.L.orc_appendix_b(C.byref(self.s), self._pc(p), C.byref(mp), _ptr(c2), _ptr(coef), _ptr(na), _ptr(ra), C.byref(res))
        return res

    def simulate_1f1b(self, p, mp, c2, coef, n, r) -> SimResult:
        """Event simulation of the 1F1B schedule for a given plan (layers n and recomputation levels r per stage)."""
        res = SimResult()
        na = np.zeros(MAX_PP, np.uint8); ra = np.zeros(MAX_PP, np.uint8)
        na[:len(n)] = n; ra[:len(r)] = r
        self.L.orc_simulate_1f1b(C.byref(self.s), self._pc(p), C.byref(mp), _ptr(c2), _ptr(coef), _ptr(na), _ptr(ra), C.byref(res))
        return res

    def bruteforce(self, p, mp, rc_mask, c2, coef, i, j):
        cnt = C.c_uint64()
        v = self.L.orc_bruteforce(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2), _ptr(coef),
                                  C.c_int(i), C.c_int(j), C.byref(cnt))
        return int(v), int(cnt.value)

    def multiset_count(self, cnt, sat=(1 << 64) - 1) -> int:
        a = np.asarray(cnt, np.int32)
        return int(self.L.orc_multiset_count(_ptr(a), C.c_int(len(a)), C.c_uint64(sat)))

    def unrank_multiset(self, cnt, idx):
        a = np.asarray(cnt, np.int32); PP = int(a.sum())
        seq = np.zeros(MAX_PP, np.uint8)
        rc = self.L.orc_unrank_multiset(_ptr(a), C.c_int(len(a)), C.c_int(PP), C.c_uint64(idx), _ptr(seq))
        return None if rc != 0 else seq[:PP].copy()

    def rank_multiset(self, cnt, seq) -> int:
        a = np.asarray(cnt, np.int32); sq = np.ascontiguousarray(np.asarray(seq, np.uint8))
        return int(self.L.orc_rank_multiset(_ptr(a), C.c_int(len(a)), C.c_int(len(sq)), _ptr(sq)))

    # ---- whole candidates ------------------------------------------------------------
    def eval_index(self, index: int, tables: bool = False):
        p = self.find_pconf(index)
        PP = int(self.pconfs["PP"][p])
        pl = Plan()
        dp = np.zeros((PP + 1, self.N + 1), np.int64) if tables else None
        ch = np.zeros((PP + 1, self.N + 1), np.uint8) if tables else None
        rc = self.L.orc_eval_index(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(self.n_pconf), C.c_uint64(index),
                                   C.byref(pl), _ptr(dp) if tables else None, _ptr(ch) if tables else None)
        assert rc == 0
        return plan_to_dict(pl), dp, ch

    def search(self, first: int = 0, count: Optional[int] = None):
        """Exhaustive evaluation of candidates [first, first+count): costs, bottlenecks, best plan."""
        if count is None:
            count = self.n_cand - first
        costs = np.zeros(count, np.int64); bn = np.zeros(count, np.int64)
        best = Plan(); feas = C.c_uint64()
        rc = self.L.orc_search(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(self.n_pconf), C.c_uint64(first),
                               C.c_uint64(count), _ptr(costs), _ptr(bn), C.byref(best), C.byref(feas))
        assert rc == 0
        return costs, bn, (plan_to_dict(best) if best.res.T_iter < INF else None), int(feas.value)

    def search_pconfs(self, p_first: int = 0, p_stride: int = 1, threads: int = 1, want_costs: bool = False):
        """All candidates of every `p_stride`-th configuration, configurations spread over `threads`
        OpenMP threads.  Returns (n evaluated, best cost, best index[, costs, bottlenecks])."""
        done = C.c_uint64(); bc = C.c_int64(); bi = C.c_uint64()
        costs = np.full(self.n_cand, -1, np.int64) if want_costs else None
        bn = np.full(self.n_cand, -1, np.int64) if want_costs else None
        try:
            omp = C.CDLL("libgomp.so.1")
            omp.omp_set_num_threads(C.c_int(threads))
        except OSError:
            pass
        self.L.orc_search_pconfs(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(self.n_pconf), C.c_uint64(p_first),
                                 C.c_uint64(p_stride), C.byref(done), C.byref(bc), C.byref(bi),
                                 _ptr(costs) if want_costs else None, _ptr(bn) if want_costs else None)
        if want_costs:
            return int(done.value), int(bc.value), int(bi.value), costs, bn
        return int(done.value), int(bc.value), int(bi.value)

    def search_pconfs_plans(self, p_first: int = 0, p_stride: int = 1, threads: int = 1):
        """search_pconfs with every candidate's partition and recomputation levels ([n_cand][MAX_PP] uint8 each;
        rows of candidates outside the selected configurations stay zero)."""
        done = C.c_uint64(); bc = C.c_int64(); bi = C.c_uint64()
        costs = np.full(self.n_cand, -1, np.int64); bn = np.full(self.n_cand, -1, np.int64)
        parts = np.zeros((self.n_cand, MAX_PP), np.uint8); levels = np.zeros((self.n_cand, MAX_PP), np.uint8)
        try:
            C.CDLL("libgomp.so.1").omp_set_num_threads(C.c_int(threads))
        except OSError:
            pass
        self.L.orc_search_pconfs_plans(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(self.n_pconf), C.c_uint64(p_first),
                                       C.c_uint64(p_stride), C.byref(done), C.byref(bc), C.byref(bi), _ptr(costs), _ptr(bn),
                                       _ptr(parts), _ptr(levels))
        return int(done.value), costs, bn, parts, levels

    # ---- refinement --------------------------------------------------------------------
    def candidate_refined(self, p, mp, rc_mask, c2, coef) -> Result:
        res = Result()
        self.L.orc_candidate_refined(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2), _ptr(coef),
                                     C.byref(res))
        return res

    def eval_index_refined(self, index: int) -> dict:
        p = self.find_pconf(index)
        n_rc = len(self.pb.rc_masks)
        local = index - int(self.pconfs["offset"][p])
        mp = self.decode(p, local // n_rc)
        c2, _, coef, _ = self.layer_costs(p)
        res = self.candidate_refined(p, mp, int(self.pb.rc_masks[local % n_rc]), c2, coef)
        PP = int(self.pconfs["PP"][p])
        return dict(T_iter=int(res.T_iter), bottleneck=int(res.bottleneck), T_pipe=int(res.T_pipe), T_sync=int(res.T_sync),
                    T_opt=int(res.T_opt), n=[int(x) for x in res.n[:PP]], r=[int(x) for x in res.r[:PP]],
                    c=[int(x) for x in res.c[:PP]], PP=PP, M=int(self.pconfs["M"][p]))

    def bruteforce_sum(self, p, mp, rc_mask, c2, coef, i, j, limit) -> int:
        return int(self.L.orc_bruteforce_sum(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2),
                                             _ptr(coef), C.c_int(i), C.c_int(j), C.c_int64(limit)))

    def search_pconfs_refined(self, p_first: int = 0, p_stride: int = 1, threads: int = 1, want_costs: bool = True):
        self.L.orc_set_refine(C.c_int(1))
        try:
            return self.search_pconfs(p_first, p_stride, threads, want_costs)
        finally:
            self.L.orc_set_refine(C.c_int(0))

    # ---- exact optimum of the pipeline term -----------------------------------------------------
    def eval_index_exact(self, index: int) -> dict:
        p = self.find_pconf(index)
        n_rc = len(self.pb.rc_masks)
        local = index - int(self.pconfs["offset"][p])
        mp = self.decode(p, local // n_rc)
        rc = int(self.pb.rc_masks[local % n_rc])
        c2, _, coef, _ = self.layer_costs(p)
        res, passes = Result(), C.c_int64()
        self.L.orc_candidate_exact(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc), _ptr(c2), _ptr(coef),
                                   C.byref(res), C.byref(passes))
        PP = int(self.pconfs["PP"][p])
        brute = int(self.L.orc_bruteforce_pipe(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc), _ptr(c2), _ptr(coef)))
        return dict(T_iter=int(res.T_iter), bottleneck=int(res.bottleneck), T_pipe=int(res.T_pipe), T_sync=int(res.T_sync),
                    T_opt=int(res.T_opt), n=[int(x) for x in res.n[:PP]], r=[int(x) for x in res.r[:PP]],
                    c=[int(x) for x in res.c[:PP]], PP=PP, M=int(self.pconfs["M"][p]), passes=int(passes.value),
                    brute_pipe=brute)

    def search_pconfs_exact(self, p_first: int = 0, p_stride: int = 1, threads: int = 1, want_costs: bool = True):
        self.L.orc_set_refine(C.c_int(2))
        try:
            return self.search_pconfs(p_first, p_stride, threads, want_costs)
        finally:
            self.L.orc_set_refine(C.c_int(0))

    # ---- joint recurrence over the device state ----------------------------------------------
    def joint_bottleneck(self, p: int, rc_mask: int, c2=None, coef=None) -> int:
        if c2 is None:
            c2, _, coef, _ = self.layer_costs(p)
        return int(self.L.orc_joint_bottleneck(C.byref(self.s), self._pc(p), C.c_uint32(rc_mask), _ptr(c2), _ptr(coef)))

    # ---- fp64 mode ---------------------------------------------------------------------
    def candidate_f64(self, p, mp, rc_mask, c2f, coef, coeff) -> ResultF:
        res = ResultF()
        self.L.orc_candidate_f64(C.byref(self.s), self._pc(p), C.byref(mp), C.c_uint32(rc_mask), _ptr(c2f), _ptr(coef),
                                 _ptr(coeff), C.byref(res))
        return res

    def eval_index_f64(self, index: int) -> dict:
        p = self.find_pconf(index)
        n_rc = len(self.pb.rc_masks)
        local = index - int(self.pconfs["offset"][p])
        mp = self.decode(p, local // n_rc)
        _, c2f, coef, coeff = self.layer_costs(p)
        res = self.candidate_f64(p, mp, int(self.pb.rc_masks[local % n_rc]), c2f, coef, coeff)
        PP = int(self.pconfs["PP"][p])
        return dict(T_iter=res.T_iter, bottleneck=res.bottleneck, T_pipe=res.T_pipe, T_sync=res.T_sync, T_opt=res.T_opt,
                    n=[int(x) for x in res.n[:PP]], r=[int(x) for x in res.r[:PP]], c=[float(x) for x in res.c[:PP]])

    def search_pconfs_f64(self, p_first: int = 0, p_stride: int = 1, threads: int = 1):
        """fp64-mode costs, bottlenecks and partitions of every candidate of every p_stride-th configuration."""
        done = C.c_uint64()
        costs = np.full(self.n_cand, -1.0, np.float64); bn = np.full(self.n_cand, -1.0, np.float64)
        parts = np.zeros((self.n_cand, MAX_PP), np.uint8)
        try:
            C.CDLL("libgomp.so.1").omp_set_num_threads(C.c_int(threads))
        except OSError:
            pass
        self.L.orc_search_pconfs_f64(C.byref(self.s), _ptr(self.pconfs), C.c_uint64(self.n_pconf), C.c_uint64(p_first),
                                     C.c_uint64(p_stride), C.byref(done), _ptr(costs), _ptr(bn), _ptr(parts))
        return int(done.value), costs, bn, parts
