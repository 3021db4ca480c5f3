"""Seeded synthetic planning problems (inputs only).

This module produces the *inputs* of the planner: a model description, a cluster
inventory, "profiled" lookup tables and the search options.  The paper obtains the
tables by profiling real accelerators (Sec. 3.3, "compute table", "communication
primitive table", "memory calibration"); here they are synthesised from a seed so that
both the CPU oracle and the CUDA path can be fed the same numbers.

Nothing of the method's arithmetic lives here (no cost formula, no enumeration, no
dynamic program): a `Problem` is plain data.  Neither `oracle/` nor the CUDA package is
imported from this module, and each of them marshals a `Problem` on its own.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List

import numpy as np

DENSE, MOE = 0, 1
MASK64 = (1 << 64) - 1


class SplitMix64:
    """splitmix64 counter-based generator; `u()` returns a double in [0, 1)."""

    def __init__(self, seed: int):
        self.state = seed & MASK64

    def next(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & MASK64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
        return z ^ (z >> 31)

    def u(self) -> float:
        return (self.next() >> 11) * (2.0 ** -53)


@dataclass
class Problem:
    """Plain-data planning problem.  All arrays are C-contiguous numpy arrays."""

    name: str
    # ---- model (Sec. 3.2 "Input": N, S, H, E, k and training hyper-parameters)
    N: int
    S: int
    H: int
    E: int
    k: int
    n_shared: int
    F_dense: int
    F_exp: int
    nq: int
    nkv: int
    V: int
    beta: float          # bytes per element
    GB: int              # global batch
    kind: np.ndarray     # [N] uint8, DENSE / MOE
    # ---- cluster (device-type triples (P_h, C_h, B_h) and inventory {m_h})
    P: np.ndarray            # [T] int64, peak GFLOP/s of the type
    C: np.ndarray            # [T] int64, memory capacity in bytes
    node_size: np.ndarray    # [T] int32, devices per node of that type
    bw_intra: np.ndarray     # [T] float64, bytes/ns inside a node
    node_type: np.ndarray    # [n_nodes] int32
    node_bw_inter: np.ndarray  # [n_nodes] float64, bytes/ns of the node's uplink
    # ---- profile: index lists (position = table index)
    tp_list: np.ndarray
    cp_list: np.ndarray
    mb_list: np.ndarray
    ep_list: np.ndarray
    # ---- profile: tables, ns.  [T][ntp][ncp][nmb][N] and [T][ntp][ncp][nmb]
    tdf: np.ndarray
    tdb: np.ndarray
    tff: np.ndarray
    tfb: np.ndarray
    tpre: np.ndarray
    tpost: np.ndarray
    eta: np.ndarray      # [T]
    croute: np.ndarray   # [T] ns per token*hidden element
    kappa: float
    alpha: np.ndarray    # [3] ns per step for INTRA, INTER, CROSS
    chi: float
    rho: np.ndarray      # [nep]
    gamma: float
    ovl_tp: float
    ovl_cp: float
    ovl_dp: float
    act_coef: np.ndarray  # [2] bytes per token*hidden element, by layer kind
    capf: float
    copt: np.ndarray     # [T] ns per parameter
    cap_eff: np.ndarray  # [T] int64 usable bytes after calibration
    xi_q: np.ndarray     # [R] int32, activation factor in 1/1024
    tau_q: np.ndarray    # [R] int32, recomputed forward fraction in 1/1024
    # ---- search options
    pp_list: np.ndarray
    tpe_list: np.ndarray
    tp_max: int
    delta_q: int         # load-balance window in 1/1024; < 0 disables it
    map_cap: int         # largest multiset-permutation count that is enumerated
    rc_masks: np.ndarray  # [n_rc] uint32, allowed recompute levels per policy
    # ---- extras that are not inputs of the method (kept for inspection)
    extra: Dict[str, np.ndarray] = field(default_factory=dict)
    uniform: int = 0     # ablation: 1 = uniform layer split only (non-uniform partitioning disabled)
    het_coll: int = 0    # Pruning 3 also counts the dispatch / combine traffic of stages that span device types
    eta_q: int = 0       # Pruning 3 threshold eta in 1/1024 (2048 = the paper's default 2); <= 0 disables it
    # communication-primitive table: link efficiency by message size (empty: efficiency 1 everywhere)
    fsize: np.ndarray = field(default_factory=lambda: np.zeros(0, np.float64))     # [n] bytes, ascending
    feff: np.ndarray = field(default_factory=lambda: np.zeros((3, 0), np.float64))  # [3][n] INTRA, INTER, CROSS

    @property
    def T(self) -> int:
        return int(self.P.shape[0])

    @property
    def W(self) -> int:
        return int(sum(int(self.node_size[t]) for t in self.node_type))

    def copy(self, **changes) -> "Problem":
        d = {}
        for f in self.__dataclass_fields__:
            v = getattr(self, f)
            d[f] = v.copy() if isinstance(v, np.ndarray) else (dict(v) if isinstance(v, dict) else v)
        d.update(changes)
        return Problem(**d)


def _i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _i64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int64))


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _pow2_upto(n: int) -> List[int]:
    out, v = [], 1
    while v <= n:
        out.append(v)
        v *= 2
    return out


def synth_tables(*, N, S, H, F_dense, F_exp, n_shared, nq, nkv, V, kind, P_tf, eff,
                 tp_list, cp_list, mb_list):
    """Synthetic compute tables.  time = flops / (TP*CP) / (rate * efficiency)."""
    T = len(P_tf)
    ntp, ncp, nmb = len(tp_list), len(cp_list), len(mb_list)
    phi_b_all = {1: 0.85, 2: 0.92, 4: 0.96, 8: 1.0}
    Hkv = H * nkv // nq
    tdf = np.zeros((T, ntp, ncp, nmb, N))
    tff = np.zeros((T, ntp, ncp, nmb, N))
    tpre = np.zeros((T, ntp, ncp, nmb))
    tpost = np.zeros((T, ntp, ncp, nmb))
    for h in range(T):
        rate = float(P_tf[h]) * 1.0e3           # flop per ns
        for itp, tp in enumerate(tp_list):
            for icp, cp in enumerate(cp_list):
                for ib, b in enumerate(mb_list):
                    tok = float(b) * float(S)
                    phi = (0.97 ** itp) * (0.98 ** icp) * phi_b_all.get(int(b), 1.0)
                    fl_attn = 2.0 * tok * H * (2.0 * H + 2.0 * Hkv) + 4.0 * tok * S * H
                    tpost[h, itp, icp, ib] = (6.0 * tok * H * V) / (tp * cp) / (rate * 0.5 * phi)
                    for l in range(N):
                        F = F_exp if kind[l] == MOE else F_dense
                        fl_ffn = 6.0 * tok * H * F
                        fl_sh = n_shared * 6.0 * tok * H * F_exp if kind[l] == MOE else 0.0
                        den = rate * eff[h, l] * phi
                        tff[h, itp, icp, ib, l] = fl_ffn / (tp * cp) / den
                        tdf[h, itp, icp, ib, l] = (fl_attn + fl_ffn + fl_sh) / (tp * cp) / den
    return tdf, 2.0 * tdf, tff, 2.0 * tff, tpre, tpost


def _build(name, seed, *, N, S, H, E, k, n_shared, F_dense, F_exp, nq, nkv, V, GB, kind,
           P_tf, C_gb, node_size, bw_intra, node_type, bw_inter_fixed, bw_inter_random,
           zipf_alpha, mb_list, rc_masks, delta_q, map_cap) -> Problem:
    T = len(P_tf)
    rng = SplitMix64(seed)
    # draw 1: per-type, per-layer efficiencies U[0.4, 0.7]
    eff = np.zeros((T, N))
    for h in range(T):
        for l in range(N):
            eff[h, l] = 0.4 + 0.3 * rng.u()
    # draw 2: Zipf expert loads, shuffled over the experts (Fisher-Yates)
    w = np.array([(r + 1.0) ** (-zipf_alpha) for r in range(E)])
    w = w / w.sum()
    perm = list(range(E))
    for i in range(E - 1, 0, -1):
        j = int(rng.u() * (i + 1))
        perm[i], perm[j] = perm[j], perm[i]
    load = np.zeros(E)
    for r in range(E):
        load[perm[r]] = w[r]
    # draw 3: per-node uplink bandwidth (only where the config asks for it)
    n_nodes = len(node_type)
    if bw_inter_random:
        node_bw = np.array([25.0 + 25.0 * rng.u() for _ in range(n_nodes)])
    else:
        node_bw = np.full(n_nodes, float(bw_inter_fixed))

    max_node = int(min(node_size))
    tp_list = [v for v in (1, 2, 4, 8) if v <= max_node]
    cp_list = [1, 2, 4, 8]
    tpe_list = list(tp_list)
    ep_list = [v for v in _pow2_upto(E) if E % v == 0]
    pp_list = [v for v in _pow2_upto(min(N, 32))]

    tdf, tdb, tff, tfb, tpre, tpost = synth_tables(
        N=N, S=S, H=H, F_dense=F_dense, F_exp=F_exp, n_shared=n_shared, nq=nq, nkv=nkv, V=V,
        kind=kind, P_tf=P_tf, eff=eff, tp_list=tp_list, cp_list=cp_list, mb_list=mb_list)

    rho_val = float(load.max() / (load.sum() / E))
    usable = 0.9
    cap_eff = [int(np.floor(float(C_gb[h]) * (2 ** 30) * usable / (1.0 + 0.02 * h))) for h in range(T)]
    return Problem(
        name=name, N=N, S=S, H=H, E=E, k=k, n_shared=n_shared, F_dense=F_dense, F_exp=F_exp,
        nq=nq, nkv=nkv, V=V, beta=2.0, GB=GB, kind=np.ascontiguousarray(np.asarray(kind, np.uint8)),
        P=_i64([int(p) * 1000 for p in P_tf]), C=_i64([int(c) * (2 ** 30) for c in C_gb]),
        node_size=_i32(node_size), bw_intra=_f64(bw_intra), node_type=_i32(node_type),
        node_bw_inter=_f64(node_bw),
        tp_list=_i32(tp_list), cp_list=_i32(cp_list), mb_list=_i32(mb_list), ep_list=_i32(ep_list),
        tdf=_f64(tdf), tdb=_f64(tdb), tff=_f64(tff), tfb=_f64(tfb), tpre=_f64(tpre), tpost=_f64(tpost),
        eta=_f64([0.95 - 0.05 * h for h in range(T)]),
        croute=_f64([2.0 * E / (0.3 * float(P_tf[h]) * 1.0e3) for h in range(T)]),
        kappa=float(k), alpha=_f64([2000.0, 8000.0, 12000.0]), chi=0.7,
        rho=_f64([rho_val] * len(ep_list)), gamma=0.5, ovl_tp=1.0, ovl_cp=0.25, ovl_dp=0.5,
        act_coef=_f64([34.0, 34.0 + 4.0 * k]), capf=1.0,
        copt=_f64([4.8 / float(P_tf[h]) for h in range(T)]), cap_eff=_i64(cap_eff),
        xi_q=_i32([1024, 64]), tau_q=_i32([0, 1024]),
        pp_list=_i32(pp_list), tpe_list=_i32(tpe_list), tp_max=max_node,
        delta_q=delta_q, map_cap=map_cap, rc_masks=np.ascontiguousarray(np.asarray(rc_masks, np.uint32)),
        extra={"eff": eff, "expert_load": load},
    )


def _nodes(counts) -> List[int]:
    out: List[int] = []
    for t, c in enumerate(counts):
        out += [t] * c
    return out


def tiny(window: bool = False) -> Problem:
    """Config 1: 16 MoE layers, 8 devices in 2 nodes of 4, two device types."""
    return _build("tiny", 0, N=16, S=2048, H=1024, E=8, k=2, n_shared=0, F_dense=4096, F_exp=4096,
                  nq=8, nkv=8, V=32000, GB=64, kind=[MOE] * 16,
                  P_tf=[400, 200], C_gb=[80, 40], node_size=[4, 4], bw_intra=[400.0, 400.0],
                  node_type=_nodes([1, 1]), bw_inter_fixed=25.0, bw_inter_random=False,
                  zipf_alpha=1.2, mb_list=[1, 2, 4, 8], rc_masks=[0b11],
                  delta_q=205 if window else -1, map_cap=1 << 40)


def small() -> Problem:
    """Config 2: 32 MoE layers, 32 devices in 4 nodes of 8, three device types."""
    return _build("small", 1, N=32, S=4096, H=2048, E=64, k=8, n_shared=0, F_dense=1024, F_exp=1024,
                  nq=16, nkv=8, V=32000, GB=256, kind=[MOE] * 32,
                  P_tf=[400, 300, 150], C_gb=[80, 64, 32], node_size=[8, 8, 8],
                  bw_intra=[900.0, 400.0, 200.0], node_type=_nodes([2, 1, 1]),
                  bw_inter_fixed=50.0, bw_inter_random=False, zipf_alpha=1.2,
                  mb_list=[1, 2, 4, 8], rc_masks=[0b11], delta_q=205, map_cap=2048)


def mixtral() -> Problem:
    """Config 3: Mixtral-8x7B shape on 64 devices, two device types split 32/32."""
    return _build("mixtral", 2, N=32, S=4096, H=4096, E=8, k=2, n_shared=0, F_dense=14336,
                  F_exp=14336, nq=32, nkv=8, V=32000, GB=512, kind=[MOE] * 32,
                  P_tf=[400, 250], C_gb=[80, 64], node_size=[8, 8], bw_intra=[900.0, 300.0],
                  node_type=_nodes([4, 4]), bw_inter_fixed=50.0, bw_inter_random=False,
                  zipf_alpha=1.2, mb_list=[1, 2, 4, 8], rc_masks=[0b11], delta_q=205, map_cap=2048)


def dsv2() -> Problem:
    """Config 4: DeepSeek-V2-like shape (first layer dense) on 256 devices, four types."""
    return _build("dsv2", 3, N=60, S=4096, H=5120, E=160, k=6, n_shared=2, F_dense=12288,
                  F_exp=1536, nq=128, nkv=128, V=102400, GB=1024, kind=[DENSE] + [MOE] * 59,
                  P_tf=[400, 300, 200, 150], C_gb=[80, 64, 48, 32], node_size=[8, 8, 8, 8],
                  bw_intra=[900.0, 600.0, 400.0, 200.0], node_type=_nodes([12, 8, 8, 4]),
                  bw_inter_fixed=50.0, bw_inter_random=True, zipf_alpha=1.4,
                  mb_list=[1, 2, 4, 8], rc_masks=[0b11], delta_q=205, map_cap=2048)


def stress() -> Problem:
    """Config 5: 96 MoE layers on 1024 devices in 128 nodes, four types in uneven counts."""
    return _build("stress", 4, N=96, S=8192, H=8192, E=256, k=8, n_shared=0, F_dense=2048,
                  F_exp=2048, nq=64, nkv=8, V=128000, GB=2048, kind=[MOE] * 96,
                  P_tf=[400, 300, 250, 150], C_gb=[80, 64, 48, 32], node_size=[8, 8, 8, 8],
                  bw_intra=[900.0, 600.0, 400.0, 200.0], node_type=_nodes([64, 32, 16, 16]),
                  bw_inter_fixed=50.0, bw_inter_random=False, zipf_alpha=1.2,
                  mb_list=[1, 2, 4], rc_masks=[0b01, 0b11], delta_q=205, map_cap=2048)


CONFIGS = {"tiny": tiny, "small": small, "mixtral": mixtral, "dsv2": dsv2, "stress": stress}


def make_problem(name: str, **kw) -> Problem:
    return CONFIGS[name](**kw)


def random_small(seed: int, *, N: int = 8, T: int = 2, nodes_per_type=(1, 1), node_size: int = 2,
                 window: bool = False, tight_memory: bool = True, first_dense: bool = False) -> Problem:
    """Small randomised problem for brute-force and property tests.

    Capacities are drawn so that the memory constraint is active for part of the candidates
    (some spans need recomputation, some are infeasible)."""
    rng = SplitMix64(0xC0FFEE ^ (seed * 7919))
    P_tf = sorted([int(100 + 50 * int(rng.u() * 7)) for _ in range(T)], reverse=True)
    C_gb = [4096 for _ in range(T)]
    kind = [MOE] * N
    if first_dense:
        kind[0] = DENSE
    pr = _build(f"rand{seed}", seed + 1000, N=N, S=1024, H=512, E=4, k=2, n_shared=0, F_dense=2048,
                F_exp=1024, nq=4, nkv=2, V=8000, GB=16, kind=kind, P_tf=P_tf, C_gb=C_gb,
                node_size=[node_size] * T, bw_intra=[float(200 + 100 * h) for h in range(T)],
                node_type=_nodes(list(nodes_per_type)), bw_inter_fixed=25.0, bw_inter_random=True,
                zipf_alpha=1.2, mb_list=[1, 2, 4], rc_masks=[0b01, 0b11],
                delta_q=205 if window else -1, map_cap=1 << 40)
    if tight_memory:
        # capacities of a few hundred MB: at this model size some stage spans fit as they are, some
        # only with recomputation and some not at all
        base = [400, 200, 300, 250]
        pr.cap_eff[:] = [int(base[h % 4] * 1.0e6 * (0.9 + 0.3 * rng.u())) for h in range(T)]
    return pr


def blank(*, N, S, H, E, k, GB, P_tf, C_gb, node_size, nodes_per_type, tp_list=(1,), cp_list=(1,),
          mb_list=(1,), ep_list=(1,), pp_list=(1,), tpe_list=(1,), kind=None, n_shared=0, F_dense=4096,
          F_exp=4096, nq=8, nkv=8, V=32000, R=1) -> Problem:
    """Problem skeleton with all-zero tables and neutral coefficients, for hand-written examples.

    Neutral means: eta = 1, kappa = 1, rho = 1, gamma = 0, zero latencies, unit bandwidths,
    overlap factors 1, no recomputation levels beyond "off", window off, huge capacities."""
    T = len(P_tf)
    kind = [MOE] * N if kind is None else kind
    ntp, ncp, nmb = len(tp_list), len(cp_list), len(mb_list)
    z5 = np.zeros((T, ntp, ncp, nmb, N))
    z4 = np.zeros((T, ntp, ncp, nmb))
    xi = [1024, 64, 32, 16][:R]
    tau = [0, 1024, 1024, 1024][:R]
    return Problem(
        name="blank", N=N, S=S, H=H, E=E, k=k, n_shared=n_shared, F_dense=F_dense, F_exp=F_exp, nq=nq,
        nkv=nkv, V=V, beta=2.0, GB=GB, kind=np.ascontiguousarray(np.asarray(kind, np.uint8)),
        P=_i64([int(p) * 1000 for p in P_tf]), C=_i64([int(c) * (2 ** 30) for c in C_gb]),
        node_size=_i32(node_size), bw_intra=_f64([1.0] * T), node_type=_i32(_nodes(list(nodes_per_type))),
        node_bw_inter=_f64([1.0] * sum(nodes_per_type)),
        tp_list=_i32(tp_list), cp_list=_i32(cp_list), mb_list=_i32(mb_list), ep_list=_i32(ep_list),
        tdf=z5.copy(), tdb=z5.copy(), tff=z5.copy(), tfb=z5.copy(), tpre=z4.copy(), tpost=z4.copy(),
        eta=_f64([1.0] * T), croute=_f64([0.0] * T), kappa=1.0, alpha=_f64([0.0, 0.0, 0.0]), chi=1.0,
        rho=_f64([1.0] * len(ep_list)), gamma=0.0, ovl_tp=1.0, ovl_cp=1.0, ovl_dp=1.0,
        act_coef=_f64([0.0, 0.0]), capf=0.0, copt=_f64([0.0] * T),
        cap_eff=_i64([int(c) * (2 ** 30) for c in C_gb]), xi_q=_i32(xi), tau_q=_i32(tau),
        pp_list=_i32(pp_list), tpe_list=_i32(tpe_list), tp_max=max(list(tp_list) + list(tpe_list)),
        delta_q=-1, map_cap=1 << 40, rc_masks=np.ascontiguousarray(np.asarray([(1 << R) - 1], np.uint32)),
    )


def with_link_efficiency_table(pb: Problem, seed: int = 7, n: int = 8) -> Problem:
    """The same problem with a synthetic communication-primitive table: link efficiency rising with the
    message size (64 KiB .. 8 GiB, factor 8 between sizes) towards 0.75-0.97, lower for slower link classes,
    with a seeded wiggle so that the interpolation segments have different slopes."""
    rng = SplitMix64(0xF00D ^ (seed * 104729))
    out = pb.copy()
    out.fsize = np.ascontiguousarray(np.array([65536.0 * 8.0 ** i for i in range(n)], np.float64))
    top = [0.97, 0.9, 0.75]
    eff = np.zeros((3, n), np.float64)
    for c in range(3):
        for i in range(n):
            ramp = (i + 1.0) / (n + 1.0)
            eff[c, i] = min(1.0, max(0.05, top[c] * (0.35 + 0.65 * ramp) + 0.03 * (rng.u() - 0.5)))
    out.feff = np.ascontiguousarray(eff)
    return out
