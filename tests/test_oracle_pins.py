"""Pins of the CPU oracle against things that are not the oracle itself:
hand-computed values (tests/golden), closed forms, invariants and brute force."""
import itertools
import json
import math
import os

import numpy as np
import pytest

from gen import problems
from gen.problems import DENSE, MOE
from oracle import Oracle, INF, COEF, NCOEF, Mapping
from hand_examples import e8_problem, e9_problem, e10_problem

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


# --------------------------------------------------------------------------------------
# input generator
# --------------------------------------------------------------------------------------
def test_splitmix64_published_vectors():
    r = problems.SplitMix64(0)
    assert [r.next() for _ in range(3)] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    r = problems.SplitMix64(1234567)
    assert [r.next() for _ in range(2)] == [6457827717110365317, 3203168211198807973]


def test_generator_is_deterministic_and_in_range():
    a, b = problems.tiny(), problems.tiny()
    for f in ("tdf", "tff", "tpost", "rho", "cap_eff"):
        assert np.array_equal(getattr(a, f), getattr(b, f))
    eff = a.extra["eff"]
    assert eff.min() >= 0.4 and eff.max() < 0.7
    assert abs(a.extra["expert_load"].sum() - 1.0) < 1e-12
    assert (a.tdf >= a.tff).all() and (a.tff > 0).all()


# --------------------------------------------------------------------------------------
# hand-computed examples
# --------------------------------------------------------------------------------------
def e1_problem():
    pb = problems.blank(N=4, S=2048, H=1024, E=4, k=2, GB=4, P_tf=[400, 200], C_gb=[100000, 100000],
                        node_size=[1, 1], nodes_per_type=[1, 1], pp_list=(2,))
    tdf_a = np.array([900000.0, 1000000.0, 1100000.0, 1000000.0])
    tff_a = np.array([500000.0, 600000.0, 700000.0, 600000.0])
    for h, sc in ((0, 1.0), (1, 2.0)):
        pb.tdf[h, 0, 0, 0] = sc * tdf_a
        pb.tff[h, 0, 0, 0] = sc * tff_a
        pb.tdb[h, 0, 0, 0] = 2 * sc * tdf_a
        pb.tfb[h, 0, 0, 0] = 2 * sc * tff_a
    pb.eta[:] = [1.0, 0.8]
    pb.croute[:] = [0.01, 0.02]
    pb.kappa = 2.0
    pb.rho[:] = 1.5
    pb.gamma = 0.5
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.node_bw_inter[:] = 25.0
    pb.bw_intra[:] = 400.0
    pb.chi = 0.7
    return pb


def test_e1_two_device_example():
    g = gold("e1_two_device_pp2.json")["expect"]
    o = Oracle(e1_problem())
    assert o.n_pconf == 1 and o.n_cand == 2
    c2, c2f, coef, _ = o.layer_costs(0)
    assert c2[0, :, 0].tolist() == g["qf_A"] and c2[0, :, 1].tolist() == g["qb_A"]
    assert c2[1, :, 0].tolist() == g["qf_B"] and c2[1, :, 1].tolist() == g["qb_B"]
    assert abs(c2f[0, 0, 0] - 1670971.52) < 1e-6 and abs(c2f[1, 0, 1] - 7933886.08) < 1e-6
    assert coef[1, COEF["KP2P_CROSS"] + 0] == g["kp2p_cross"] and coef[0, COEF["KP2P_CROSS"] + 1] == g["kp2p_cross"]
    plan0, dp, ch = o.eval_index(0, tables=True)
    ab = g["map_AB"]
    assert plan0["mask"] == [1, 2]
    assert dp[1, 1:4].tolist() == ab["dp_row1"] and dp[2, 2:5].tolist() == ab["dp_row2"]
    assert ch[2, 2:5].tolist() == ab["ch_row2"]
    assert plan0["n"] == ab["n"] and plan0["bottleneck"] == ab["bottleneck"] and plan0["T_iter"] == ab["T_iter"]
    assert dp[0, 0] == 0 and dp[1, 0] == INF and dp[2, 1] == INF and dp[1, 4] == INF
    plan1, _, _ = o.eval_index(1)
    ba = g["map_BA"]
    assert plan1["mask"] == [2, 1]
    assert plan1["n"] == ba["n"] and plan1["bottleneck"] == ba["bottleneck"] and plan1["T_iter"] == ba["T_iter"]
    costs, bn, best, feas = o.search()
    assert best["index"] == g["best_map"] and feas == 2 and costs.tolist() == [ab["T_iter"], ba["T_iter"]]


def test_e1_heterogeneous_communication_pruning():
    g = gold("e1_two_device_pp2.json")["expect"]["pruning3"]
    for eta_q, want in g.items():
        pb = e1_problem()
        pb.eta_q = int(eta_q)
        costs, bn, best, feas = Oracle(pb).search()
        assert costs.tolist() == [INF if w == "INF" else w for w in want]
        assert bn.tolist() == [17288745, 18542094]           # the bottleneck itself is not touched by the rule
        assert (best is None) == (want == ["INF", "INF"])


def test_e1_fp64_mode_hand_values():
    g = gold("e1_two_device_pp2.json")["expect"]["fp64"]
    o = Oracle(e1_problem())
    for idx, key in ((0, "map_AB"), (1, "map_BA")):
        r = o.eval_index_f64(idx)
        assert r["n"] == g[key]["n"]
        assert r["T_iter"] == pytest.approx(g[key]["T_iter"], rel=1e-12)
        assert r["c"] == pytest.approx(g[key]["c"], rel=1e-12)
        assert r["bottleneck"] == pytest.approx(max(g[key]["c"]), rel=1e-12)


def test_fp64_mode_tracks_integer_mode_within_rounding():
    """Each of the <= 2N+PP rounded terms moves a time by at most 0.5 ns, times M for the bottleneck term."""
    for pb in (problems.tiny(), problems.random_small(2, N=9, T=2, nodes_per_type=(2, 2), node_size=2)):
        o = Oracle(pb)
        ci, bi, _, _ = o.search()
        done, cf, bf, parts = o.search_pconfs_f64(0, 1, threads=2)
        assert done == o.n_cand
        fin = ci < INF
        assert np.array_equal(fin, np.isfinite(cf)) and np.array_equal(bi < INF, np.isfinite(bf))
        M = np.repeat(o.pconfs["M"].astype(np.float64), o.pconfs["nmap"].astype(np.int64) * len(pb.rc_masks))
        # rounding can also flip a near-tie between partitions, so allow a relative slack as well
        assert (np.abs(bf[fin] - bi[fin]) <= (2 * pb.N + 2) * 0.5 + 1e-6 * bi[fin]).all()
        assert (np.abs(cf[fin] - ci[fin]) <= M[fin] * (2 * pb.N + 34) + 2e-3 * ci[fin]).all()
        assert (parts[fin].sum(axis=1) == pb.N).all()


def test_e2_dispatch_volume_and_primitive_tie():
    g = gold("e2_dispatch_ep2.json")["expect"]
    pb = e1_problem()
    pb = problems.blank(N=4, S=2048, H=1024, E=4, k=2, GB=4, P_tf=[400], C_gb=[100000], node_size=[2],
                        nodes_per_type=[1], pp_list=(1,), ep_list=(2,))
    src = e1_problem()
    for f in ("tdf", "tdb", "tff", "tfb"):
        getattr(pb, f)[0] = getattr(src, f)[0]
    pb.croute[:] = 0.01
    pb.kappa, pb.gamma = 2.0, 0.5
    pb.rho[:] = 1.5
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.bw_intra[:] = 400.0
    o = Oracle(pb)
    assert o.n_pconf == 1 and int(o.pconfs["EP"][0]) == 2 and int(o.pconfs["DP"][0]) == 2
    c2, _, _, _ = o.layer_costs(0)
    assert c2[0, 0].tolist() == [g["qf0"], g["qb0"]]


def e4_problem(k=1):
    pb = problems.blank(N=2, S=2048, H=1024, E=4, k=k, GB=8, P_tf=[400], C_gb=[100000], node_size=[4],
                        nodes_per_type=[2], pp_list=(1,), tp_list=(1, 2), cp_list=(1, 2), ep_list=(1, 2),
                        tpe_list=(1,), kind=[DENSE, MOE], n_shared=1, F_dense=4096, F_exp=2048, nq=8, nkv=4)
    pb.tdf[0, 1, 1, 0] = [1000000.0, 900000.0]
    pb.tdb[0, 1, 1, 0] = [2000000.0, 1800000.0]
    pb.tff[0, 1, 1, 0] = [300000.0, 400000.0]
    pb.tfb[0, 1, 1, 0] = [600000.0, 800000.0]
    pb.tpre[0, 1, 1, 0] = 1234.4
    pb.tpost[0, 1, 1, 0] = 5678.5
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.bw_intra[:] = 400.0
    pb.node_bw_inter[:] = [25.0, 30.0]          # the slower uplink of the type counts
    pb.chi, pb.ovl_tp, pb.ovl_cp, pb.ovl_dp = 0.7, 1.0, 0.25, 0.5
    pb.eta[:] = 0.8
    pb.kappa, pb.gamma, pb.capf = 2.0, 0.5, 1.0
    pb.rho[:] = 1.5
    pb.croute[:] = 0.01
    pb.act_coef[:] = [34.0, 38.0]
    pb.copt[:] = 0.012
    return pb


def _find(o, **kw):
    hits = [p for p in range(o.n_pconf) if all(int(o.pconfs[k][p]) == v for k, v in kw.items())]
    assert len(hits) == 1, hits
    return hits[0]


def test_e4_collectives_memory_and_sync_terms():
    g = gold("e4_collectives_memory_sync.json")["expect"]
    o = Oracle(e4_problem(k=1))
    p = _find(o, PP=1, TP=2, CP=2, EP=2, TPE=1, b=1)
    assert int(o.pconfs["DP"][p]) == 2 and int(o.pconfs["EDP"][p]) == 4 and int(o.pconfs["M"][p]) == 4
    c2, _, coef, _ = o.layer_costs(p)
    assert c2[0, 0].tolist() == g["dense"] and c2[0, 1].tolist() == g["moe_k1"]
    row = coef[0]
    assert [row[COEF["MW"]], row[COEF["MW"] + 1]] == g["mw"]
    assert [row[COEF["MA"]], row[COEF["MA"] + 1]] == g["ma"]
    assert row[COEF["MX"]] == g["mx"] and row[COEF["MPRE"]] == g["mpre"] and row[COEF["MPOST"]] == g["mpre"]
    assert [row[COEF["SBW"]], row[COEF["SBW"] + 1]] == g["sbw"] and row[COEF["SLAT"]] == g["slat"]
    assert [row[COEF["OPT"]], row[COEF["OPT"] + 1]] == g["opt"]
    assert [row[COEF["KP2P_INTRA"]], row[COEF["KP2P_INTER"]], row[COEF["KP2P_CROSS"]]] == g["kp2p"]
    assert row[COEF["KPRE"]] == g["kpre"] and row[COEF["KPOST"]] == g["kpost"]
    o4 = Oracle(e4_problem(k=4))
    c2k4, _, _, _ = o4.layer_costs(_find(o4, PP=1, TP=2, CP=2, EP=2, TPE=1, b=1))
    assert c2k4[0, 1, 0] == g["moe_k4_fwd"]


def test_e3_minimal_recompute_level():
    g = gold("e3_minimal_recompute.json")["expect"]
    GiB = 1 << 30
    pb = problems.blank(N=6, S=2048, H=1024, E=4, k=2, GB=4, P_tf=[400], C_gb=[40], node_size=[1],
                        nodes_per_type=[2], pp_list=(2,), R=2)
    o = Oracle(pb)
    assert int(o.pconfs["M"][0]) == 4
    mp = o.decode(0, 0)
    c2 = np.zeros((1, 6, 2), np.int64)
    c2[0, :, 0], c2[0, :, 1] = 100, 200
    coef = np.zeros((1, NCOEF), np.int64)
    coef[0, COEF["MW"] + MOE] = 10 * GiB
    coef[0, COEF["MA"] + MOE] = 2 * GiB
    val = lambda x: INF if x == "INF" else x
    assert list(o.stage_cost(0, mp, 0b11, c2, coef, 2, 3, 6)) == g["s2_3layers"]
    assert list(o.stage_cost(0, mp, 0b11, c2, coef, 1, 0, 3)) == g["s1_3layers"]
    assert o.stage_cost(0, mp, 0b01, c2, coef, 1, 0, 3)[0] == val(g["s1_3layers_mask1"])
    assert o.stage_cost(0, mp, 0b11, c2, coef, 1, 0, 4)[0] == val(g["s1_4layers"])
    assert o.stage_cost(0, mp, 0b01, c2, coef, 1, 0, 4)[0] == val(g["s1_4layers"])


# --------------------------------------------------------------------------------------
# special cases of the cost formulas
# --------------------------------------------------------------------------------------
def test_eq2_reduces_to_dense_plus_router_when_nothing_is_sharded():
    # EP = TPE = 1, eta = kappa = rho = 1: the expert term equals the FFN it replaces
    pb = problems.blank(N=3, S=1024, H=512, E=4, k=2, GB=2, P_tf=[100], C_gb=[1000], node_size=[1],
                        nodes_per_type=[1], pp_list=(1,))
    pb.tdf[0, 0, 0, 0] = [7000.0, 8000.5, 9000.25]
    pb.tff[0, 0, 0, 0] = [3000.0, 1000.0, 2000.0]
    pb.tdb[:] = 2 * pb.tdf
    pb.tfb[:] = 2 * pb.tff
    pb.croute[:] = 0.001
    o = Oracle(pb)
    _, c2f, _, _ = o.layer_costs(0)
    tr = 0.001 * 1024 * 512
    assert np.allclose(c2f[0, :, 0], pb.tdf[0, 0, 0, 0] + tr, rtol=1e-15)
    assert np.allclose(c2f[0, :, 1], pb.tdb[0, 0, 0, 0] + 2 * tr, rtol=1e-15)


def test_collective_model_closed_forms():
    # world 1 costs nothing; doubling the bytes doubles the bandwidth part; the link class switches
    # exactly when the group extent exceeds the node size
    def tp_comm(TP, node, bytes_scale=1.0, alpha=0.0):
        pb = problems.blank(N=1, S=1024, H=int(512 * bytes_scale), E=4, k=2, GB=64, P_tf=[100], C_gb=[1000],
                            node_size=[node], nodes_per_type=[8 // node], pp_list=(1,), tp_list=(TP,),
                            kind=[DENSE], nq=8, nkv=8)
        pb.alpha[:] = alpha
        pb.bw_intra[:] = 100.0
        pb.node_bw_inter[:] = 10.0
        o = Oracle(pb)
        _, c2f, _, _ = o.layer_costs(0)
        return c2f[0, 0, 0]
    assert tp_comm(1, 8) == 0.0
    base = tp_comm(2, 8)
    assert base == 4 * (1024 * 512 * 2.0 * 0.5) / 100.0          # 2 blocks x 2 collectives x D*(w-1)/w / bw
    assert tp_comm(2, 8, bytes_scale=2.0) == 2 * base
    assert tp_comm(4, 4) == 4 * (1024 * 512 * 2.0 * 0.75) / 100.0   # extent 4 = node size: intra
    assert tp_comm(8, 4) == 4 * (1024 * 512 * 2.0 * 0.875) / 10.0   # extent 8 > node size: inter
    assert tp_comm(2, 8, alpha=500.0) == base + 4 * 500.0


def test_ep1_has_no_dispatch_volume():
    pb = problems.blank(N=1, S=1024, H=512, E=4, k=2, GB=2, P_tf=[100], C_gb=[1000], node_size=[2],
                        nodes_per_type=[1], pp_list=(1,), ep_list=(1, 2))
    pb.tdf[:] = 1000.0
    pb.alpha[:] = 100.0
    pb.capf = 1.0
    o = Oracle(pb)
    p1, p2 = _find(o, EP=1), _find(o, EP=2)
    a, _, ca, _ = o.layer_costs(p1)
    b, _, cb, _ = o.layer_costs(p2)
    assert a[0, 0, 0] == 1000                                    # no dispatch, no latency at EP=1
    # k = EP = 2: all-to-all and all-gather volumes tie: D = 1024*512*2*2*(1/2) = 1048576
    assert b[0, 0, 0] == 1000 + 2 * (100 + 1048576)
    assert ca[0, COEF["MX"]] == 1024 * 4 * 4                     # only routing metadata at EP=1
    assert cb[0, COEF["MX"]] == 2 * 1048576 + 1024 * 4 * 4


# --------------------------------------------------------------------------------------
# enumeration, mapping, unranking
# --------------------------------------------------------------------------------------
def _brute_enumeration(pb):
    m = [0] * pb.T
    for t in pb.node_type:
        m[t] += int(pb.node_size[t])
    W = sum(m)
    rows = []
    for PP, TP, CP, EP, TPE, b in itertools.product(pb.pp_list, pb.tp_list, pb.cp_list, pb.ep_list,
                                                     pb.tpe_list, pb.mb_list):
        PP, TP, CP, EP, TPE, b = map(int, (PP, TP, CP, EP, TPE, b))
        if PP > pb.N or W % PP:
            continue
        G = W // PP
        if G % (TP * CP) or G % (EP * TPE) or pb.E % EP or TP > pb.tp_max or TPE > pb.tp_max:
            continue
        if pb.nq % TP or pb.nkv % TP or pb.S % (2 * CP):
            continue
        DP = G // (TP * CP)
        if pb.GB % (DP * b):
            continue
        rows.append((PP, TP, CP, DP, EP, TPE, b, pb.GB // (DP * b)))
    return rows


@pytest.mark.parametrize("name,npc,ncand", [("tiny", 508, 1432), ("small", 2392, 76368), ("mixtral", 3180, 36264),
                                            ("dsv2", 6536, 1945344), ("stress", 7783, 2410320)])
def test_enumeration_matches_filtered_product(name, npc, ncand):
    pb = problems.make_problem(name)
    o = Oracle(pb)
    rows = _brute_enumeration(pb)
    got = [tuple(int(o.pconfs[f][p]) for f in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M")) for p in range(o.n_pconf)]
    assert got == rows                                    # same set, same (lexicographic loop) order
    assert (o.n_pconf, o.n_cand) == (npc, ncand)
    W = pb.W
    for (PP, TP, CP, DP, EP, TPE, b, M) in rows:
        assert PP * TP * CP * DP == W and (TP * CP * DP) % (EP * TPE) == 0 and M * DP * b == pb.GB
    offs = o.pconfs["offset"].astype(np.int64)
    sizes = o.pconfs["nmap"].astype(np.int64) * len(pb.rc_masks)
    assert offs[0] == 0 and np.array_equal(offs[1:], np.cumsum(sizes)[:-1]) and offs[-1] + sizes[-1] == o.n_cand


def test_multiset_unranking_against_sorted_permutations():
    o = Oracle(problems.tiny())
    for cnt in ([2, 2], [1, 1], [3, 1, 2], [2, 0, 1, 2], [4, 4], [1, 2, 1, 1]):
        seqs = sorted(set(itertools.permutations([h for h, c in enumerate(cnt) for _ in range(c)])))
        n = o.multiset_count(cnt)
        PP = sum(cnt)
        assert n == len(seqs) == math.factorial(PP) // math.prod(math.factorial(c) for c in cnt)
        for i, s in enumerate(seqs):
            got = o.unrank_multiset(cnt, i)
            assert tuple(got.tolist()) == s
            assert o.rank_multiset(cnt, got) == i
        assert o.unrank_multiset(cnt, n) is None
    assert o.multiset_count([16, 8, 4, 4]) == math.factorial(32) // (math.factorial(16) * math.factorial(8) * 24 * 24)
    assert o.multiset_count([16, 8, 4, 4], sat=2049) == 2049     # saturates instead of overflowing
    assert o.multiset_count([16, 16]) == math.comb(32, 16)


def _device_line_decode(pb, PP, mode, map_idx):
    """Independent device-by-device construction of a mapping: list every device, slice per stage."""
    T = pb.T
    lines = {h: [] for h in range(T)}                      # per type: (type, node id) per device
    for n, t in enumerate(pb.node_type):
        lines[int(t)] += [(int(t), n)] * int(pb.node_size[t])
    W = sum(len(v) for v in lines.values())
    G = W // PP
    stages = []
    if mode == 0:
        cnt = [len(lines[h]) // G for h in range(T)]
        seqs = sorted(set(itertools.permutations([h for h, c in enumerate(cnt) for _ in range(c)])))
        seq = seqs[map_idx]
        used = [0] * T
        for h in seq:
            stages.append(lines[h][used[h] * G:(used[h] + 1) * G])
            used[h] += 1
    else:
        sigma = list(itertools.permutations(range(T)))[map_idx]
        line = [d for h in sigma for d in lines[h]]
        stages = [line[s * G:(s + 1) * G] for s in range(PP)]
    masks = [sum(1 << h for h in set(d[0] for d in st)) for st in stages]
    cls = [0]
    for s in range(1, PP):
        a, b = stages[s - 1][-1], stages[s][0]
        cls.append(2 if a[0] != b[0] else (0 if a[1] == b[1] else 1))
    return masks, cls


@pytest.mark.parametrize("name", ["tiny", "small", "mixtral", "dsv2", "stress"])
def test_decode_matches_device_by_device_construction(name):
    pb = problems.make_problem(name)
    o = Oracle(pb)
    seen = set()
    rng = np.random.default_rng(5)
    for p in range(o.n_pconf):
        PP, mode, nmap = int(o.pconfs["PP"][p]), int(o.pconfs["mode"][p]), int(o.pconfs["nmap"][p])
        if (PP, mode) in seen:
            continue
        seen.add((PP, mode))
        idxs = range(nmap) if nmap <= 80 else sorted(set([0, 1, nmap - 1] + rng.integers(0, nmap, 40).tolist()))
        for mi in idxs:
            mp = o.decode(p, mi)
            masks, cls = _device_line_decode(pb, PP, mode, mi)
            assert list(mp.mask[:PP]) == masks, (PP, mode, mi)
            assert list(mp.cls[1:PP]) == cls[1:], (PP, mode, mi)
        assert o.decode(p, nmap) is None
    assert {m for (_, m) in seen} == ({0, 1} if name != "mixtral" else {0, 1} & {m for (_, m) in seen})


def test_window_bounds_hand_example():
    # stages on types with 300/100/100/300 TFLOP/s, N=32, delta=0.2 (205/1024):
    # shares 3/8 and 1/8 of 32 layers = 12 and 4; bounds floor(0.7998*12)=9, ceil(1.2002*12)=15, floor(3.19)=3, ceil(4.80)=5
    pb = problems.blank(N=32, S=1024, H=512, E=4, k=2, GB=8, P_tf=[300, 100], C_gb=[1000, 1000], node_size=[1, 1],
                        nodes_per_type=[2, 2], pp_list=(4,))
    pb.delta_q = 205
    o = Oracle(pb)
    for mi in range(int(o.pconfs["nmap"][0])):
        mp = o.decode(0, mi)
        lo, hi = o.window(0, mp)
        for s in range(4):
            assert (lo[s], hi[s]) == ((9, 15) if mp.mask[s] == 1 else (3, 5))


# --------------------------------------------------------------------------------------
# recurrence, partition, objective
# --------------------------------------------------------------------------------------
def _canonical_partition_by_bruteforce(o, p, mp, rc, c2, coef, PP, N):
    """Partition defined without the recurrence: the last stage starts at the smallest k for which
    the exhaustive optimum is reached, then the same rule on the prefix."""
    n, j = [], N
    for i in range(PP, 0, -1):
        target, _ = o.bruteforce(p, mp, rc, c2, coef, i, j)
        pick = None
        for k in range(i - 1, j):
            left, _ = o.bruteforce(p, mp, rc, c2, coef, i - 1, k)
            c, _ = o.stage_cost(p, mp, rc, c2, coef, i, k, j)
            if left < INF and max(left, c) == target:
                pick = k
                break
        assert pick is not None
        n.append(j - pick)
        j = pick
    return n[::-1]


def test_bottleneck_equals_exhaustive_minimum_on_every_tiny_candidate():
    pb = problems.tiny()
    o = Oracle(pb)
    costs, bn, best, feas = o.search()
    n_checked = 0
    for p in range(o.n_pconf):
        PP = int(o.pconfs["PP"][p])
        c2, _, coef, _ = o.layer_costs(p)
        for mi in range(int(o.pconfs["nmap"][p])):
            mp = o.decode(p, mi)
            idx = int(o.pconfs["offset"][p]) + mi
            v, cnt = o.bruteforce(p, mp, 0b11, c2, coef, PP, pb.N)
            assert cnt == math.comb(pb.N - 1, PP - 1)
            assert v == bn[idx], (p, mi)
            n_checked += 1
    assert n_checked == 1432


@pytest.mark.parametrize("seed", range(6))
def test_recurrence_partition_and_objective_on_random_problems(seed):
    pb = problems.random_small(seed, N=7 + seed % 3, T=2, nodes_per_type=(2, 2), node_size=2,
                               window=(seed % 2 == 1), first_dense=(seed % 3 == 0))
    o = Oracle(pb)
    costs, bn, best, feas = o.search()
    assert 0 < feas < o.n_cand                      # some candidates infeasible, some feasible
    n_rc = len(pb.rc_masks)
    saw_recompute = False
    for idx in range(0, o.n_cand, 3):
        p = o.find_pconf(idx)
        PP, M = int(o.pconfs["PP"][p]), int(o.pconfs["M"][p])
        local = idx - int(o.pconfs["offset"][p])
        mp = o.decode(p, local // n_rc)
        rc = int(pb.rc_masks[local % n_rc])
        c2, _, coef, _ = o.layer_costs(p)
        v, _ = o.bruteforce(p, mp, rc, c2, coef, PP, pb.N)
        assert v == bn[idx]
        plan, dp, ch = o.eval_index(idx, tables=True)
        assert plan["T_iter"] == costs[idx]
        if v >= INF:
            assert costs[idx] == INF
            continue
        assert plan["n"] == _canonical_partition_by_bruteforce(o, p, mp, rc, c2, coef, PP, pb.N)
        assert sum(plan["n"]) == pb.N and min(plan["n"]) >= 1
        # closed form: what is left after the per-stage sum is (M-1) x the slowest stage
        assert plan["T_pipe"] - sum(plan["c"]) == (M - 1) * max(plan["c"]) and max(plan["c"]) == v
        assert plan["T_iter"] == plan["T_pipe"] + plan["T_sync"] + plan["T_opt"]
        # independent feasibility check of the returned partition (Eq. 1 constraint)
        a = 0
        lo, hi = o.window(p, mp)
        for s, (n, r) in enumerate(zip(plan["n"], plan["r"])):
            kinds = pb.kind[a:a + n]
            Wb = sum(int(coef[0, COEF["MW"] + kd]) for kd in kinds) + (int(coef[0, COEF["MX"]]) if (kinds == MOE).any() else 0)
            Wb += int(coef[0, COEF["MPRE"]]) if s == 0 else 0
            Wb += int(coef[0, COEF["MPOST"]]) if s == PP - 1 else 0
            A = min(M, PP - s) * sum(int(coef[0, COEF["MA"] + kd]) for kd in kinds)
            cap = min(int(pb.cap_eff[h]) for h in range(pb.T) if plan["mask"][s] >> h & 1)
            assert Wb + (int(pb.xi_q[r]) * A) // 1024 <= cap
            assert (rc >> r) & 1
            for r_lower in range(r):                    # minimal level: every lower allowed level must not fit
                if (rc >> r_lower) & 1:
                    assert Wb + (int(pb.xi_q[r_lower]) * A) // 1024 > cap
            assert lo[s] <= n <= hi[s]
            saw_recompute |= r > 0
            a += n
    assert saw_recompute
    # argmin: lowest cost, lowest index on ties
    fin = np.where(costs < INF)[0]
    assert best["index"] == int(fin[np.argmin(costs[fin])]) and best["T_iter"] == int(costs.min())


def _uniform_problem(N, PP_list, W, M_gb):
    pb = problems.blank(N=N, S=1024, H=512, E=4, k=2, GB=M_gb, P_tf=[100], C_gb=[100000], node_size=[1],
                        nodes_per_type=[W], pp_list=PP_list)
    pb.tdf[:] = 5000.0
    pb.tdb[:] = 10000.0
    pb.tff[:] = 1000.0
    pb.tfb[:] = 2000.0
    pb.bw_intra[:] = 1.0e15          # stage-to-stage transfers cost nothing, so stages differ only by layers
    pb.node_bw_inter[:] = 1.0e15
    return pb


def test_uniform_cluster_and_layers_give_even_split_and_closed_form():
    for N, PP, GB in ((12, 4, 8), (16, 8, 8), (9, 3, 5)):
        o = Oracle(_uniform_problem(N, (PP,), PP, GB))
        plan, _, _ = o.eval_index(0)
        assert plan["n"] == [N // PP] * PP
        c = (N // PP) * 15000
        assert plan["bottleneck"] == c and plan["T_pipe"] == (plan["M"] + PP - 1) * c and plan["M"] == GB


def _simulate_1f1b(f, b, M):
    """Event simulation of the 1F1B schedule (warm-up forwards, alternate, cool-down backwards)
    with zero transfer time; returns the makespan."""
    PP = len(f)
    order = []
    for s in range(PP):
        warm = min(PP - s - 1, M)
        ops = [("F", m) for m in range(warm)]
        nf, nb = warm, 0
        while nb < M:
            if nf < M:
                ops.append(("F", nf)); nf += 1
            ops.append(("B", nb)); nb += 1
        order.append(ops)
    done = {}
    t_free = [0.0] * PP
    ptr = [0] * PP
    remaining = sum(len(o) for o in order)
    while remaining:
        progressed = False
        for s in range(PP):
            while ptr[s] < len(order[s]):
                kind, m = order[s][ptr[s]]
                dep = ("F", m, s - 1) if kind == "F" and s > 0 else (("B", m, s + 1) if kind == "B" and s < PP - 1 else None)
                if kind == "B" and s == PP - 1:
                    dep = ("F", m, s)
                if dep is not None and dep not in done:
                    break
                start = max(t_free[s], done.get(dep, 0.0))
                t_free[s] = start + (f[s] if kind == "F" else b[s])
                done[(kind, m, s)] = t_free[s]
                ptr[s] += 1
                remaining -= 1
                progressed = True
        assert progressed
    return max(t_free)


def test_closed_form_equals_1f1b_simulation_for_uniform_stages():
    for PP, M, f, b in ((4, 8, 3.0, 6.0), (2, 5, 1.0, 2.0), (8, 8, 2.0, 5.0), (3, 1, 1.0, 1.0)):
        assert _simulate_1f1b([f] * PP, [b] * PP, M) == (M + PP - 1) * (f + b)
    # non-uniform stages: no equality is claimed; on this instance the closed form sum + (M-1)*max
    # over-estimates the simulated makespan slightly, and the bottleneck stage alone bounds it from below
    sim = _simulate_1f1b([3.0, 4.0, 3.0], [6.0, 8.0, 6.0], 6)
    assert 6 * 12.0 <= sim <= 30.0 + (6 - 1) * 12.0


# --------------------------------------------------------------------------------------
# monotonicity and feasibility
# --------------------------------------------------------------------------------------
def _all_costs(pb):
    o = Oracle(pb)
    costs, bn, _, _ = o.search()
    n_rc = len(pb.rc_masks)
    single = np.repeat(o.pconfs["PP"] == 1, o.pconfs["nmap"].astype(np.int64) * n_rc)
    return costs, bn, single


@pytest.mark.parametrize("field,factor", [("tdf", 1.1), ("tdb", 1.1), ("alpha", 1.5), ("croute", 2.0), ("rho", 1.2),
                                          ("copt", 1.5), ("bw_intra", 0.5), ("node_bw_inter", 0.5),
                                          ("cap_eff", 0.02)])
def test_costs_are_monotone_in_added_load(field, factor):
    """The bottleneck (a min over partitions of a max of monotone stage costs) can only grow when load is
    added.  The iteration time is the bottleneck-optimal partition's sum + (M-1)*max, so it is monotone
    wherever the partition cannot move (one stage), and for terms outside the recurrence (optimizer)."""
    pb = problems.tiny()
    c0, b0, single = _all_costs(pb)
    pb2 = pb.copy()
    arr = getattr(pb2, field)
    if arr.dtype == np.int64:
        arr[:] = (arr * factor).astype(np.int64)
    else:
        arr[:] = arr * factor
    c1, b1, _ = _all_costs(pb2)
    assert (b1 >= b0).all()
    assert (c1[single] >= c0[single]).all()
    if field == "copt":
        assert (b1 == b0).all() and (c1 >= c0).all() and (c1 > c0).any()
    else:
        assert (b1 > b0).any()


def test_adding_a_layer_never_lowers_the_bottleneck():
    pb = problems.tiny()
    c0, b0, single = _all_costs(pb)
    N = pb.N
    pb2 = pb.copy(N=N + 1, kind=np.append(pb.kind, np.uint8(MOE)))
    for f in ("tdf", "tdb", "tff", "tfb"):
        a = getattr(pb, f)
        setattr(pb2, f, np.ascontiguousarray(np.concatenate([a, a[..., -1:]], axis=-1)))
    c1, b1, _ = _all_costs(pb2)
    assert b1.shape == b0.shape and (b1 >= b0).all() and (c1[single] > c0[single]).all()


def test_infeasible_memory_plans_are_never_chosen():
    pb = problems.small()
    o = Oracle(pb)
    costs, bn, best, feas = o.search()
    assert feas < o.n_cand and (costs[bn >= INF] == INF).all() and best["T_iter"] < INF
    # shrinking every capacity far enough makes everything infeasible
    pb2 = pb.copy()
    pb2.cap_eff[:] = 1 << 20
    c2, _, best2, feas2 = Oracle(pb2).search(0, 2000)
    assert feas2 == 0 and best2 is None and (c2 == INF).all()


# --------------------------------------------------------------------------------------
# refinement: smallest stage-cost sum among the bottleneck-optimal partitions
# --------------------------------------------------------------------------------------
def _refined_partition_by_bruteforce(o, p, mp, rc, c2, coef, PP, N, limit):
    n, j = [], N
    for i in range(PP, 0, -1):
        target = o.bruteforce_sum(p, mp, rc, c2, coef, i, j, limit)
        pick = None
        for k in range(i - 1, j):
            left = o.bruteforce_sum(p, mp, rc, c2, coef, i - 1, k, limit)
            c, _ = o.stage_cost(p, mp, rc, c2, coef, i, k, j)
            if left < INF and c <= limit and left + c == target:
                pick = k
                break
        assert pick is not None
        n.append(j - pick)
        j = pick
    return n[::-1]


@pytest.mark.parametrize("seed", range(4))
def test_refinement_is_the_exhaustive_minimum_sum_under_the_bottleneck(seed):
    pb = problems.random_small(seed, N=8 + seed % 3, T=2, nodes_per_type=(2, 2), node_size=2, window=(seed % 2 == 1),
                               first_dense=(seed % 2 == 0))
    o = Oracle(pb)
    costs, bn, _, _ = o.search()
    n_rc = len(pb.rc_masks)
    changed = 0
    for idx in range(0, o.n_cand, 5):
        p = o.find_pconf(idx)
        PP, M = int(o.pconfs["PP"][p]), int(o.pconfs["M"][p])
        local = idx - int(o.pconfs["offset"][p])
        mp = o.decode(p, local // n_rc)
        rc = int(pb.rc_masks[local % n_rc])
        c2, _, coef, _ = o.layer_costs(p)
        ref = o.eval_index_refined(idx)
        if bn[idx] >= INF:
            assert ref["T_iter"] == INF
            continue
        plain, _, _ = o.eval_index(idx)
        assert ref["bottleneck"] == bn[idx] == max(ref["c"])                 # the bottleneck stays optimal
        best_sum = o.bruteforce_sum(p, mp, rc, c2, coef, PP, pb.N, int(bn[idx]))
        assert sum(ref["c"]) == best_sum <= sum(plain["c"])
        assert ref["n"] == _refined_partition_by_bruteforce(o, p, mp, rc, c2, coef, PP, pb.N, int(bn[idx]))
        assert ref["T_pipe"] == best_sum + (M - 1) * int(bn[idx]) <= plain["T_pipe"]
        assert ref["T_iter"] == ref["T_pipe"] + ref["T_sync"] + ref["T_opt"]
        # no cheaper sum exists even one unit below the bottleneck limit that still reaches B*
        assert o.bruteforce_sum(p, mp, rc, c2, coef, PP, pb.N, int(bn[idx]) - 1) == INF
        changed += ref["n"] != plain["n"]


def test_refinement_changes_some_partitions_and_never_raises_the_pipeline_time():
    o = Oracle(problems.tiny())
    c0, b0, _, _ = o.search()
    done, bc, bi, c1, b1 = o.search_pconfs_refined(0, 1, threads=2)
    assert np.array_equal(b0, b1)
    moved = [i for i in np.nonzero(c0 != c1)[0]]
    assert len(moved) > 0
    for i in moved[:20]:
        plain, _, _ = o.eval_index(int(i))
        ref = o.eval_index_refined(int(i))
        assert ref["T_pipe"] <= plain["T_pipe"] and ref["n"] != plain["n"]


# --------------------------------------------------------------------------------------
# joint recurrence over the device state (Sec. 3.5 / Algorithm 1 form)
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("make", [lambda: problems.tiny(), lambda: problems.tiny(window=True),
                                  lambda: problems.small().copy(map_cap=1 << 40, mb_list=np.array([4], np.int32)),
                                  lambda: problems.random_small(3, N=9, T=3, nodes_per_type=(2, 1, 1), node_size=2, window=True)])
def test_joint_device_state_recurrence_equals_minimum_over_enumerated_sequences(make):
    """One DP over (layers placed, stages of each type used, last type) must return the minimum, over every
    stage-type sequence, of the per-sequence bottleneck that the enumeration + per-candidate DP gives."""
    pb = make()
    if pb.name == "small":
        for f in ("tdf", "tdb", "tff", "tfb", "tpre", "tpost"):
            setattr(pb, f, np.ascontiguousarray(np.take(getattr(pb, f), [2], axis=3)))
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=4, want_costs=True)
    n_rc = len(pb.rc_masks)
    checked = 0
    for p in range(o.n_pconf):
        off, nmap, mode = int(o.pconfs["offset"][p]), int(o.pconfs["nmap"][p]), int(o.pconfs["mode"][p])
        c2, _, coef, _ = o.layer_costs(p)
        for rc in range(n_rc):
            jb = o.joint_bottleneck(p, int(pb.rc_masks[rc]), c2, coef)
            if mode == 0:
                assert jb == bn[off + rc: off + nmap * n_rc: n_rc].min(), (p, rc)
                checked += 1
            else:
                G, m = int(o.pconfs["G"][p]), [0] * pb.T
                for t in pb.node_type:
                    m[t] += int(pb.node_size[t])
                assert (jb == -1) == any(x % G for x in m)
    assert checked > 20


# --------------------------------------------------------------------------------------
# exact optimum of the pipeline term sum + (M-1) max by the upward sweep of the stage-cost limit
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("make,step", [(lambda: problems.tiny(), 2), (lambda: problems.tiny(window=True), 3),
                                       (lambda: problems.random_small(1, N=9, T=2, nodes_per_type=(2, 2), node_size=2), 4),
                                       (lambda: problems.random_small(6, N=8, T=3, nodes_per_type=(2, 1, 1), node_size=2,
                                                                      window=True, first_dense=True), 7)])
def test_limit_sweep_reaches_the_exhaustive_optimum_of_the_pipeline_term(make, step):
    pb = make()
    o = Oracle(pb)
    costs, bn, _, _ = o.search()
    improved = swept = 0
    for idx in range(0, o.n_cand, step):
        ex = o.eval_index_exact(idx)
        if bn[idx] >= INF:
            assert ex["T_iter"] == INF
            continue
        ref = o.eval_index_refined(idx)
        assert ex["T_pipe"] == ex["brute_pipe"]                      # the optimum over ALL partitions
        assert ex["T_pipe"] == sum(ex["c"]) + (ex["M"] - 1) * max(ex["c"]) <= ref["T_pipe"]
        assert sum(ex["n"]) == pb.N and ex["bottleneck"] == bn[idx] <= max(ex["c"])
        improved += ex["T_pipe"] < ref["T_pipe"]
        swept += ex["passes"] > 2
    if pb.name == "tiny":
        assert improved > 0 and swept > 0


# --------------------------------------------------------------------------------------
# Appendix B: steady-state term with the bottleneck stage's index
# --------------------------------------------------------------------------------------
def test_appendix_b_hand_values_on_the_two_device_example():
    g = gold("e5_appendix_b.json")["expect"]
    o = Oracle(e1_problem())
    c2, _, coef, _ = o.layer_costs(0)
    for idx, key in ((0, "map_AB"), (1, "map_BA")):
        plan, _, _ = o.eval_index(idx)
        assert plan["n"] == g[key]["n"]
        r = o.appendix_b(0, o.decode(0, idx), c2, coef, plan["n"], plan["r"])
        assert (r.s_max, r.T_edge, r.T_middle, r.T_iter) == (g[key]["s_max"], g[key]["T_edge"], g[key]["T_middle"], g[key]["T_iter"])
        assert r.T_edge == sum(plan["c"])                  # T_edge is the summed stage cost of the recurrence
    # fewer micro-batches than the bottleneck's index + 1: no steady-state repetitions are left
    pb = e1_problem()
    pb.GB = 2
    o2 = Oracle(pb)
    assert int(o2.pconfs["M"][0]) == 2
    c2, _, coef, _ = o2.layer_costs(0)
    r = o2.appendix_b(0, o2.decode(0, 1), c2, coef, [1, 3], [0, 0])
    assert (r.T_middle, r.T_iter) == (g["map_BA_M2"]["T_middle"], g["map_BA_M2"]["T_iter"])
    # a layer vector that does not cover the N layers is rejected
    assert o.appendix_b(0, o.decode(0, 0), c2, coef, [2, 1], [0, 0]).T_iter == INF
    assert o.appendix_b(0, o.decode(0, 0), c2, coef, [4, 0], [0, 0]).T_iter == INF


def test_appendix_b_against_the_closed_form_and_the_schedule_simulation():
    """Identities that hold for every plan: with s = s_max and M >= s + 1,
    T_appB = closed form - s * max_i c_i + sum_{i <= s} t_f,i (so it never exceeds the closed form);
    for uniform stages (f, b per micro-batch) it is (M + PP - 2)(f + b) + f, i.e. exactly b below the
    simulated 1F1B makespan (M + PP - 1)(f + b): the appendix's expression and the schedule differ by one
    backward pass of the bottleneck stage."""
    pb = problems.tiny()
    o = Oracle(pb)
    rng = np.random.default_rng(4)
    checked = 0
    for idx in rng.integers(0, o.n_cand, 400).tolist():
        plan, _, _ = o.eval_index(int(idx))
        if plan["T_iter"] >= INF:
            continue
        p = o.find_pconf(int(idx))
        c2, _, coef, _ = o.layer_costs(p)
        mp = o.decode(p, (int(idx) - int(o.pconfs["offset"][p])) // len(pb.rc_masks))
        r = o.appendix_b(p, mp, c2, coef, plan["n"], plan["r"])
        c = plan["c"]
        M, s = plan["M"], r.s_max
        assert r.T_edge == sum(c) and c[s - 1] == max(c) and all(x < max(c) for x in c[:s - 1])
        a = sum(plan["n"][:s])
        # forward time of stages 1..s: slowest member type per layer
        tf = 0
        lo = 0
        for st in range(s):
            types = [h for h in range(pb.T) if plan["mask"][st] >> h & 1]
            tf += sum(max(int(c2[h, l, 0]) for h in types) for l in range(lo, lo + plan["n"][st]))
            lo += plan["n"][st]
        assert lo == a
        assert r.T_middle == tf + max(0, M - s - 1) * max(c)
        assert (r.T_sync, r.T_opt) == (plan["T_sync"], plan["T_opt"])
        if M >= s + 1:
            assert r.T_iter == plan["T_iter"] - s * max(c) + tf and r.T_iter <= plan["T_iter"]
        checked += 1
    assert checked > 50
    for PP, M, f, b in ((4, 8, 3.0, 6.0), (2, 5, 1.0, 1.0), (8, 12, 2.0, 5.0)):
        appb = PP * (f + b) + f + (M - 1 - 1) * (f + b)           # s_max = 1 for identical stages
        assert appb == (M + PP - 2) * (f + b) + f
        assert _simulate_1f1b([f] * PP, [b] * PP, M) - appb == b


# --------------------------------------------------------------------------------------
# communication-primitive table: link efficiency by message size
# --------------------------------------------------------------------------------------
def _e1_with_table(sizes, intra, inter, cross):
    pb = e1_problem()
    pb.fsize = np.ascontiguousarray(np.array(sizes, np.float64))
    pb.feff = np.ascontiguousarray(np.array([intra, inter, cross], np.float64))
    return pb


def test_link_efficiency_table_hand_values():
    g = gold("e6_link_efficiency.json")["expect"]
    _, _, coef0, _ = Oracle(e1_problem()).layer_costs(0)
    assert coef0[0, COEF["KP2P_INTRA"]] == g["kp2p_intra_no_table"]            # 2 * (2000 + 10485.76)
    _, _, coef, _ = Oracle(_e1_with_table([1e6, 1e7], [0.5, 0.9], [0.45, 0.85], [0.4, 0.8])).layer_costs(0)
    assert coef[0, COEF["KP2P_INTRA"]] == g["kp2p_intra"]
    assert coef[1, COEF["KP2P_CROSS"] + 0] == g["kp2p_cross"] and coef[0, COEF["KP2P_CROSS"] + 1] == g["kp2p_cross"]
    _, _, coef, _ = Oracle(_e1_with_table([1e7, 1e8], [0.5, 0.9], [0.45, 0.85], [0.4, 0.8])).layer_costs(0)
    assert coef[0, COEF["KP2P_INTRA"]] == g["kp2p_intra_below"]
    _, _, coef, _ = Oracle(_e1_with_table([1e5, 1e6], [0.5, 0.9], [0.45, 0.85], [0.4, 0.8])).layer_costs(0)
    assert coef[0, COEF["KP2P_INTRA"]] == g["kp2p_intra_above"]


def test_link_efficiency_table_limits_and_monotonicity():
    """Efficiency 1 everywhere is the model without a table, bit for bit; a lower efficiency never lowers a layer
    time or a communication coefficient, and leaves the memory coefficients alone."""
    pb = problems.small()
    o0 = Oracle(pb)
    ones = problems.with_link_efficiency_table(pb)
    ones.feff = np.ones_like(ones.feff)
    o1 = Oracle(ones)
    ot = Oracle(problems.with_link_efficiency_table(pb))
    comm = [COEF[k] for k in ("KP2P_INTRA", "KP2P_INTER", "SBW")] + [COEF["KP2P_CROSS"] + q for q in range(4)] + [COEF["SBW"] + 1]
    mem = [COEF["MW"], COEF["MW"] + 1, COEF["MA"], COEF["MA"] + 1, COEF["MX"], COEF["MPRE"], COEF["MPOST"], COEF["OPT"], COEF["SLAT"]]
    grew = 0
    for p in range(0, o0.n_pconf, 37):
        a, af, ac, _ = o0.layer_costs(p)
        b, bf, bc, _ = o1.layer_costs(p)
        c, cf, cc, _ = ot.layer_costs(p)
        assert np.array_equal(a, b) and np.array_equal(af, bf) and np.array_equal(ac, bc)
        assert (c >= a).all() and (cc[:, comm] >= ac[:, comm]).all() and np.array_equal(cc[:, mem], ac[:, mem])
        grew += int((c > a).any())
    assert grew > 0


# --------------------------------------------------------------------------------------
# event simulation of the 1F1B schedule for given plans
# --------------------------------------------------------------------------------------
def _longest_path_1f1b(f, b, M):
    """The same schedule as a precedence graph: a pass ends at its duration plus the latest end among the pass
    before it on its stage and the pass that produces its input; evaluated by memoised recursion (no event loop)."""
    import functools
    import sys
    PP = len(f)
    prev_on_stage = {}
    for s in range(PP):
        warm = min(PP - s - 1, M)
        ops = [("F", m) for m in range(warm)]
        nf, nb = warm, 0
        while nb < M:
            if nf < M:
                ops.append(("F", nf)); nf += 1
            ops.append(("B", nb)); nb += 1
        for a, c in zip([None] + ops[:-1], ops):
            prev_on_stage[(c[0], s, c[1])] = None if a is None else (a[0], s, a[1])
    sys.setrecursionlimit(max(10000, 8 * PP * M + 1000))

    @functools.lru_cache(maxsize=None)
    def end(kind, s, m):
        t = 0
        p = prev_on_stage[(kind, s, m)]
        if p is not None:
            t = max(t, end(*p))
        if kind == "F" and s > 0:
            t = max(t, end("F", s - 1, m))
        if kind == "B":
            t = max(t, end("B", s + 1, m) if s < PP - 1 else end("F", s, m))
        return t + (f[s] if kind == "F" else b[s])
    return max(end("B", s, M - 1) for s in range(PP))


def test_1f1b_schedule_worked_examples_and_two_formulations_agree():
    g = gold("e7_1f1b_schedule.json")
    for case in g["cases"]:
        assert _simulate_1f1b(case["f"], case["b"], case["M"]) == case["makespan"], case["name"]
        assert _longest_path_1f1b(tuple(case["f"]), tuple(case["b"]), case["M"]) == case["makespan"], case["name"]
        c = [x + y for x, y in zip(case["f"], case["b"])]
        assert sum(c) + (case["M"] - 1) * max(c) == case["closed_form_sum_plus_M_minus_1_max"]
    rng = np.random.default_rng(12)
    for _ in range(60):
        PP, M = int(rng.integers(1, 9)), int(rng.integers(1, 12))
        f = tuple(int(x) for x in rng.integers(1, 20, PP)); b = tuple(int(x) for x in rng.integers(1, 40, PP))
        sim = _simulate_1f1b(list(f), list(b), M)
        assert sim == _longest_path_1f1b(f, b, M)
        c = [x + y for x, y in zip(f, b)]
        # the bottleneck stage alone and one trip through the pipeline bound the makespan from below, running every
        # pass one after another from above.  Eq. 4's pipeline term is neither: with unequal stages the schedule
        # can end a little after it (c = (27, 28, 42, 9), M = 8 below) as well as before it.
        assert max(M * max(c), sum(c)) <= sim <= M * sum(c)
        if PP == 1:
            assert sim == M * c[0]
        if M == 1:
            assert sim == sum(c)
    # Eq. 4's pipeline term is not an upper bound of the schedule
    f, b = (16, 11, 6, 7), (11, 17, 36, 2)
    assert [x + y for x, y in zip(f, b)] == [27, 28, 42, 9]
    assert _simulate_1f1b(list(f), list(b), 8) == _longest_path_1f1b(f, b, 8) == 401 > 106 + 7 * 42


def test_oracle_1f1b_simulation_hand_example_and_closed_forms():
    g = gold("e7_1f1b_schedule.json")["oracle_case"]
    o = Oracle(_uniform_problem(g["N"], (g["PP"],), g["PP"], g["GB"]))
    c2, _, coef, _ = o.layer_costs(0)
    r = o.simulate_1f1b(0, o.decode(0, 0), c2, coef, g["n"], [0] * g["PP"])
    assert (r.T_pipe_sim, r.T_pipe_closed) == (g["T_pipe_sim_ns"], g["T_pipe_closed_ns"])
    assert r.T_iter == r.T_pipe_sim + r.T_sync + r.T_opt
    # identical stages: the simulated schedule takes exactly Eq. 4's (M + PP - 1) c
    for N, PP, GB in ((12, 4, 8), (16, 8, 8), (9, 3, 5), (6, 1, 4), (8, 8, 1)):
        o = Oracle(_uniform_problem(N, (PP,), PP, GB))
        c2, _, coef, _ = o.layer_costs(0)
        r = o.simulate_1f1b(0, o.decode(0, 0), c2, coef, [N // PP] * PP, [0] * PP)
        c = (N // PP) * 15000
        assert r.T_pipe_sim == (GB + PP - 1) * c == r.T_pipe_closed
    # a layer vector that does not cover the N layers is rejected
    assert o.simulate_1f1b(0, o.decode(0, 0), c2, coef, [2] + [1] * 7, [0] * 8).T_iter == INF
    assert o.simulate_1f1b(0, o.decode(0, 0), c2, coef, [0] + [1] * 6 + [2], [0] * 8).T_iter == INF


def test_oracle_1f1b_simulation_against_the_python_schedule_on_searched_plans():
    """Plans the search returns for tiny and small (several types per stage, recomputation, transfer constants):
    the oracle's simulation equals the two Python formulations fed with the plan's own per-stage forward and
    backward times, respects the bounds that hold for every schedule, and shares T_sync / T_opt with Eq. 4."""
    checked = 0
    for pb in (problems.tiny(), problems.small()):
        o = Oracle(pb)
        rng = np.random.default_rng(8)
        for idx in rng.integers(0, o.n_cand, 300).tolist():
            plan, _, _ = o.eval_index(int(idx))
            if plan["T_iter"] >= INF or plan["M"] > 64:
                continue
            p = o.find_pconf(int(idx))
            c2, _, coef, _ = o.layer_costs(p)
            mp = o.decode(p, (int(idx) - int(o.pconfs["offset"][p])) // len(pb.rc_masks))
            r = o.simulate_1f1b(p, mp, c2, coef, plan["n"], plan["r"])
            tf, lo = [], 0
            for st in range(plan["PP"]):
                types = [h for h in range(pb.T) if plan["mask"][st] >> h & 1]
                tf.append(sum(max(int(c2[h, l, 0]) for h in types) for l in range(lo, lo + plan["n"][st])))
                lo += plan["n"][st]
            tb = [c - x for c, x in zip(plan["c"], tf)]
            assert all(x >= 0 for x in tb)
            sim = _simulate_1f1b(tf, tb, plan["M"])
            assert r.T_pipe_sim == sim == _longest_path_1f1b(tuple(tf), tuple(tb), plan["M"]), idx
            assert r.T_pipe_closed == plan["T_pipe"] and (r.T_sync, r.T_opt) == (plan["T_sync"], plan["T_opt"])
            assert max(plan["M"] * max(plan["c"]), sum(plan["c"])) <= r.T_pipe_sim <= plan["M"] * sum(plan["c"])
            assert r.T_iter == r.T_pipe_sim + r.T_sync + r.T_opt
            checked += 1
    assert checked > 80


# --------------------------------------------------------------------------------------
# Eq. 4's synchronisation and optimizer terms over the stages; stages that span two device types
# --------------------------------------------------------------------------------------
def _check_plan(o, index, want):
    pl, _, _ = o.eval_index(index)
    for key in ("n", "c", "bottleneck", "T_pipe", "T_sync", "T_opt", "T_iter"):
        assert pl[key] == want[key], (index, key, pl[key], want[key])
    if "r" in want:
        assert pl["r"] == want["r"]
    return pl


def test_e8_sync_and_optimizer_terms_are_the_slowest_stage_of_each():
    g = gold("e8_sync_opt_assembly.json")["expect"]
    o = Oracle(e8_problem())
    assert (o.n_pconf, o.n_cand) == (1, 6)
    assert [int(o.pconfs[k][0]) for k in ("PP", "DP", "EDP", "M", "G")] == [3, 4, 4, 4, 4]
    _, _, coef, _ = o.layer_costs(0)
    for h, name in enumerate("ABC"):
        assert [coef[h, COEF["SBW"]], coef[h, COEF["SBW"] + 1]] == g["coef"]["sbw"][name]
        assert [coef[h, COEF["OPT"]], coef[h, COEF["OPT"] + 1]] == g["coef"]["opt"][name]
        assert coef[h, COEF["SLAT"]] == g["coef"]["slat"]
        assert all(coef[h, COEF["KP2P_CROSS"] + h2] == g["coef"]["kp2p_cross"] for h2 in range(3))
    for name in ("ABC", "BAC"):
        want = g[name]
        mp = o.decode(0, want["map_idx"])
        assert [int(m).bit_length() - 1 for m in mp.mask[:3]] == ["ABC".index(ch) for ch in name]
        _check_plan(o, want["map_idx"], want)
    # the three terms are decided by three different stages in the first mapping, so none of the plausible
    # mistakes (sum over stages, the bottleneck stage's own terms, one stage for both terms) reproduces it
    a = g["ABC"]
    assert a["T_iter"] == a["T_pipe"] + a["T_sync"] + a["T_opt"]
    assert a["c"].index(a["bottleneck"]) == 0 and a["T_sync"] == 12000 + 2 * 660741 and a["T_opt"] == 3 * 352395


def test_e9_stage_spanning_two_device_types():
    g = gold("e9_mixed_type_stage.json")["expect"]
    o = Oracle(e9_problem())
    assert (o.n_pconf, o.n_cand) == (1, 2)
    assert int(o.pconfs["nmap"][0]) == 2 and int(o.pconfs["G"][0]) == 4 and int(o.pconfs["M"][0]) == 4
    c2, _, coef, _ = o.layer_costs(0)
    m = g["mem_coef"]
    assert coef[0, COEF["MW"] + MOE] == m["mw"] and coef[0, COEF["MA"] + MOE] == m["ma"]
    assert coef[0, COEF["MX"]] == m["mx"] and coef[0, COEF["MPRE"]] == m["mpre"] == coef[0, COEF["MPOST"]]
    for name in ("AB", "BA"):
        want = g[name]
        mp = o.decode(0, want["map_idx"])
        assert [int(x) for x in mp.mask[:2]] == g["masks"][name]
        assert int(mp.cls[1]) == 0                      # the boundary lies inside type A's node
        lo, hi = o.window(0, mp)
        assert [[int(lo[s]), int(hi[s])] for s in range(2)] == g["window"][name]
        pl = _check_plan(o, want["map_idx"], want)
        assert pl["mask"] == g["masks"][name]
    mp = o.decode(0, 0)
    for n2, (cost, level) in g["stage2_AB_spans"].items():
        assert o.stage_cost(0, mp, 0b11, c2, coef, 2, 8 - int(n2), 8) == (cost, level)
    # without recomputation the mixed stage holds one layer only (B's 2 GiB), which the window still allows
    assert o.stage_cost(0, mp, 0b01, c2, coef, 2, 6, 8)[0] == INF
    assert o.stage_cost(0, mp, 0b01, c2, coef, 2, 7, 8) == (1314486, 0)
    costs, _, best, _ = o.search()
    assert costs.tolist() == [g["AB"]["T_iter"], g["BA"]["T_iter"]] and best["index"] == g["best_index"]


def test_e10_dispatch_of_mixed_type_stages_in_the_heterogeneous_communication_rule():
    """Pruning 3 with the dispatch / combine traffic of stages that span device types: the coefficient, which
    stages and layers count, and the decisions around the hand-computed thresholds."""
    g = gold("e10_hetero_dispatch.json")["expect"]
    o = Oracle(e10_problem())
    assert (o.n_pconf, o.n_cand) == (1, 2)
    assert [int(o.pconfs[k][0]) for k in ("EP", "EDP", "M", "G")] == [2, 2, 4, 4]
    c2, c2f, coef, coeff = o.layer_costs(0)
    assert coef[:, COEF["KXD"]].tolist() == g["kxd"]
    assert coeff[:, COEF["KXD"]].tolist() == pytest.approx(g["kxd_f64"], rel=1e-14)
    assert c2.sum(axis=2).tolist() == [g["layer_sum"]["A"], g["layer_sum"]["B"]]
    for name in ("AB", "BA"):
        mp = o.decode(0, g[name]["map_idx"])
        assert [int(x) for x in mp.mask[:2]] == g["masks"][name] and int(mp.cls[1]) == 0
    for eta_q, want in g["pruned"].items():
        for variant in ("plain", "refined", "exact", "f64"):
            pb = e10_problem()
            pb.eta_q = int(eta_q)
            ov = Oracle(pb)
            for name, dropped in zip(("AB", "BA"), want):
                idx = g[name]["map_idx"]
                got = {"plain": lambda: ov.eval_index(idx)[0], "refined": lambda: ov.eval_index_refined(idx),
                       "exact": lambda: ov.eval_index_exact(idx), "f64": lambda: ov.eval_index_f64(idx)}[variant]()
                assert got["n"] == g[name]["n"], (eta_q, variant, name)
                if variant == "f64":
                    assert (got["T_iter"] == float("inf")) == dropped, (eta_q, variant, name)
                else:
                    assert got["bottleneck"] == g[name]["bottleneck"]
                    assert got["T_iter"] == (INF if dropped else g[name]["T_iter"]), (eta_q, variant, name)
    # the narrow reading sees no cross-type traffic here: nothing is dropped, whatever eta
    for eta_q, want in g["pruned_without_option"].items():
        pb = e10_problem()
        pb.eta_q, pb.het_coll = int(eta_q), 0
        costs, _, best, feas = Oracle(pb).search()
        assert costs.tolist() == [g["AB"]["T_iter"], g["BA"]["T_iter"]] and feas == 2 and best["index"] == 1


@pytest.mark.parametrize("make, gname, names", [(e8_problem, "e8_sync_opt_assembly.json", ("ABC", "BAC")),
                                                (e9_problem, "e9_mixed_type_stage.json", ("AB", "BA"))])
def test_every_objective_variant_assembles_sync_and_optimizer_terms_alike(make, gname, names):
    """The hand examples have one optimal partition under every objective (smallest bottleneck, smallest sum under
    it, exact pipeline term), so the refinement, the exact sweep, the fp64 mode and the post-hoc evaluators must
    report the hand-computed T_sync and T_opt as well."""
    g = gold(gname)["expect"]
    o = Oracle(make())
    c2, _, coef, _ = o.layer_costs(0)
    for name in names:
        want = g[name]
        for got in (o.eval_index_refined(want["map_idx"]), o.eval_index_exact(want["map_idx"])):
            for key in ("n", "c", "bottleneck", "T_pipe", "T_sync", "T_opt", "T_iter"):
                assert got[key] == want[key], (name, key)
        mp = o.decode(0, want["map_idx"])
        r = want.get("r", [0] * len(want["n"]))
        for res in (o.appendix_b(0, mp, c2, coef, want["n"], r), o.simulate_1f1b(0, mp, c2, coef, want["n"], r)):
            assert (int(res.T_sync), int(res.T_opt)) == (want["T_sync"], want["T_opt"])
        f = o.eval_index_f64(want["map_idx"])
        assert f["n"] == want["n"]
        for key in ("T_sync", "T_opt", "T_pipe", "T_iter"):      # fp64 mode keeps the coefficients unrounded
            assert abs(f[key] - want[key]) <= 1.0 * (len(want["n"]) + 8), (name, key, f[key])


def test_e8_fp64_mode_hand_values():
    # unrounded terms of the first mapping: sync 12000 + 2*660741.12, optimizer 3*352395.264,
    # transfers 503349.0285714...; T_pipe = 9e6 + (6e6 + x) + (7.2e6 + x) + 3*9e6 with x the transfer
    o = Oracle(e8_problem())
    f = o.eval_index_f64(0)
    x = 2.0 * (12000.0 + 4194304.0 / 17.5)
    assert f["T_sync"] == pytest.approx(1333482.24, rel=1e-13)
    assert f["T_opt"] == pytest.approx(1057185.792, rel=1e-13)
    assert f["T_pipe"] == pytest.approx(49200000.0 + 2.0 * x, rel=1e-13)
    assert f["T_iter"] == pytest.approx(49200000.0 + 2.0 * x + 1333482.24 + 1057185.792, rel=1e-13)


def test_bulk_search_with_plans_agrees_with_single_candidate_evaluation():
    """Plumbing of the bulk search that also returns partitions and levels: same values as eval_index."""
    o = Oracle(problems.tiny(window=True))
    done, costs, bn, parts, levels = o.search_pconfs_plans(0, 1, threads=2)
    assert done == o.n_cand
    for idx in range(0, o.n_cand, 13):
        pl, _, _ = o.eval_index(idx)
        assert costs[idx] == pl["T_iter"] and bn[idx] == pl["bottleneck"]
        if pl["T_iter"] < INF:
            assert parts[idx, :pl["PP"]].tolist() == pl["n"] and levels[idx, :pl["PP"]].tolist() == pl["r"]
            assert not parts[idx, pl["PP"]:].any()
        else:
            assert not parts[idx].any() and not levels[idx].any()
