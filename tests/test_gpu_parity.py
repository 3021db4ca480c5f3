"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Integer mode: layer costs, coefficients, decoded mappings, DP tables, split choices, partitions,
recomputation levels, bottlenecks, iteration times and the winning index must be bit-identical.
The unrounded fp64 layer costs must agree within 1e-9 relative (they are the same IEEE operations
in the same order, so in practice they agree exactly)."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from gen import problems  # noqa: E402
from oracle import Oracle, INF  # noqa: E402

CONFIGS = ["tiny", "small", "mixtral", "dsv2", "stress"]
NTHREADS = max(1, len(os.sched_getaffinity(0)))


@pytest.fixture(scope="module")
def hap():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    return hap


_cache = {}


def setup(hap, name, **kw):
    key = (name, tuple(sorted(kw.items())))
    if key not in _cache:
        pb = problems.make_problem(name, **kw)
        hp = hap.hap_problem_create(pb)
        hap.hap_enumerate(hp)
        _cache[key] = (pb, hp, Oracle(pb))
    return _cache[key]


@pytest.mark.parametrize("name", CONFIGS)
def test_enumeration_is_identical(hap, name):
    pb, hp, o = setup(hap, name)
    assert (hp.n_pconf, hp.n_cand) == (o.n_pconf, o.n_cand)
    got = hap.hap_get_pconfs(hp)
    for f in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M", "EDP", "G", "itp", "icp", "ib", "iep", "mode", "nmap", "offset"):
        assert np.array_equal(got[f], o.pconfs[f]), f


@pytest.mark.parametrize("name", CONFIGS)
def test_layer_costs_and_coefficients_bit_exact(hap, name):
    pb, hp, o = setup(hap, name)
    c2, coef = hap.hap_eval_layer_costs(hp)
    c2f, coeff = hap.hap_eval_layer_costs_f64(hp)
    torch.cuda.synchronize()
    c2, coef, c2f, coeff = c2.cpu().numpy(), coef.cpu().numpy(), c2f.cpu().numpy(), coeff.cpu().numpy()
    for p in range(o.n_pconf):                  # every configuration: all (configuration, type, layer) units
        e2, e2f, ecoef, ecoeff = o.layer_costs(p)
        assert np.array_equal(c2[p], e2), p
        assert np.array_equal(coef[p], ecoef), p
        assert np.allclose(c2f[p], e2f, rtol=1e-9, atol=0.0), p
        assert np.allclose(coeff[p], ecoeff, rtol=1e-9, atol=0.0), p


@pytest.mark.parametrize("name", CONFIGS)
def test_decode_matches_oracle(hap, name):
    pb, hp, o = setup(hap, name)
    n_rc = len(pb.rc_masks)
    rng = np.random.default_rng(11)
    if o.n_cand <= 80000:
        ranges = [(0, o.n_cand)]
    else:
        starts = sorted(set([0, o.n_cand - 700] + rng.integers(0, o.n_cand - 700, 30).tolist()))
        ranges = [(s, 700) for s in starts]
    for first, count in ranges:
        got = hap.hap_decode(hp, first, count)
        for q in range(0, count, 1 if count <= 2000 else 7):
            idx = first + q
            p = o.find_pconf(idx)
            local = idx - int(o.pconfs["offset"][p])
            mp = o.decode(p, local // n_rc)
            PP = int(o.pconfs["PP"][p])
            g = got[q]
            assert int(g["index"]) == idx and int(g["pconf"]) == p and int(g["PP"]) == PP
            assert int(g["map_idx"]) == local // n_rc and int(g["rc_mask"]) == int(pb.rc_masks[local % n_rc])
            assert g["mask"][:PP].tolist() == list(mp.mask[:PP]) and not g["mask"][PP:].any()
            link = [(mp.cls[s] | (mp.ha[s] << 2) | (mp.hb[s] << 4)) if s else 0 for s in range(PP)]
            assert g["link"][:PP].tolist() == link, (idx, g["link"][:PP].tolist(), link)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}),
                                     ("dsv2", {}), ("stress", {})])
def test_every_candidate_cost_and_bottleneck_bit_exact(hap, name, kw):
    """Whole candidate space, in the launch configuration the benchmark times."""
    pb, hp, o = setup(hap, name, **kw)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    torch.cuda.synchronize()
    done, costs, bn, parts, levels = o.search_pconfs_plans(0, 1, threads=NTHREADS)
    assert done == o.n_cand
    order = np.lexsort((np.arange(o.n_cand), costs))
    bc, bi = int(costs[order[0]]), int(order[0])
    got_c, got_b = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy()
    bad = np.nonzero(got_c != costs)[0]
    assert bad.size == 0, (bad[:10], got_c[bad[:10]], costs[bad[:10]])
    assert np.array_equal(got_b, bn)
    # the partition and the recomputation levels of EVERY candidate (the default kernel: the prefix tree)
    bad = np.nonzero((out["partition"].cpu().numpy() != parts).any(axis=1))[0]
    assert bad.size == 0, bad[:10]
    bad = np.nonzero((out["recompute"].cpu().numpy() != levels).any(axis=1))[0]
    assert bad.size == 0, bad[:10]
    assert (parts[costs < INF].sum(axis=1) == pb.N).all() and not parts[costs >= INF].any()
    # argmin of the device cost array: lowest cost, lowest index on ties
    am = hap.hap_argmin(hp, out["cost"]).cpu().numpy()
    assert (int(am[0]), int(am[1])) == (bc, bi)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}),
                                     ("dsv2", {}), ("stress", {})])
def test_tables_partitions_and_recompute_bit_exact(hap, name, kw):
    pb, hp, o = setup(hap, name, **kw)
    rng = np.random.default_rng(3)
    if o.n_cand <= 2000:
        ranges = [(0, o.n_cand)]
    else:
        starts = sorted(set([0, o.n_cand - 64] + rng.integers(0, o.n_cand - 64, 24).tolist()))
        ranges = [(s, 64) for s in starts]
    N = pb.N
    for first, count in ranges:
        out = hap.hap_pipeline_dp(hp, first, count, partition=True, tables=True)
        torch.cuda.synchronize()
        dp, ch = out["dp_table"].cpu().numpy(), out["choice"].cpu().numpy()
        part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
        cost, bott = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy()
        for q in range(0, count, 1 if o.n_cand <= 2000 else 5):
            plan, edp, ech = o.eval_index(first + q, tables=True)
            PP = plan["PP"]
            assert np.array_equal(dp[q, :PP + 1], edp), (first + q)
            assert np.array_equal(ch[q, :PP + 1], ech), (first + q)
            assert (dp[q, PP + 1:] == -1).all() and (ch[q, PP + 1:] == 254).all()     # rows beyond PP untouched
            assert cost[q] == plan["T_iter"] and bott[q] == plan["bottleneck"]
            if plan["T_iter"] < INF:
                assert part[q, :PP].tolist() == plan["n"] and rec[q, :PP].tolist() == plan["r"]
                assert int(part[q].sum()) == N
            else:
                assert not part[q].any() and not rec[q].any()
            assert not part[q, PP:].any()


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}),
                                     ("dsv2", {}), ("stress", {})])
def test_search_best_returns_the_oracle_plan(hap, name, kw):
    pb, hp, o = setup(hap, name, **kw)
    plan, stats = hap.hap_search_best(hp)
    done, bc, bi = o.search_pconfs(0, 1, threads=NTHREADS)
    assert (plan["T_iter"], plan["index"]) == (bc, bi)
    eplan, _, _ = o.eval_index(bi)
    for key in ("PP", "TP", "CP", "DP", "EP", "TPE", "b", "M", "n", "r", "mask", "rc_mask", "bottleneck", "T_pipe", "T_sync", "T_opt"):
        assert plan[key] == eplan[key], key
    assert stats["n_candidates"] == o.n_cand and stats["n_evaluated"] + stats["n_pruned"] == o.n_cand
    assert sum(plan["n"]) == pb.N


def test_sub_ranges_ragged_edges_and_errors(hap):
    pb, hp, o = setup(hap, "small")
    costs, bn, best, feas = o.search(1000, 3001)
    out = hap.hap_pipeline_dp(hp, 1000, 3001)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs)
    plan, stats = hap.hap_search_range(hp, 1000, 3001)
    assert plan["index"] == best["index"] and plan["T_iter"] == best["T_iter"] and stats["n_evaluated"] == 3001
    for key in ("n", "r", "mask", "bottleneck", "T_pipe", "T_sync", "T_opt"):
        assert plan[key] == best[key], key
    # single candidate, last candidate, empty range
    one = hap.hap_pipeline_dp(hp, o.n_cand - 1, 1)
    torch.cuda.synchronize()
    assert int(one["cost"].cpu()[0]) == o.eval_index(o.n_cand - 1)[0]["T_iter"]
    hap.hap_pipeline_dp(hp, 5, 0)
    with pytest.raises(hap.HapError) as e:
        hap.hap_pipeline_dp(hp, o.n_cand - 1, 2)
    assert e.value.name == "HAP_E_RANGE"
    with pytest.raises(hap.HapError):
        hap.hap_search_range(hp, 0, 0)


def test_all_infeasible_and_bad_descriptors(hap):
    pb = problems.small()
    pb.cap_eff[:] = 1 << 20
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    with pytest.raises(hap.HapError) as e:
        hap.hap_search_range(hp, 0, 5000)
    assert e.value.name == "HAP_E_INFEASIBLE"
    out = hap.hap_pipeline_dp(hp, 0, 5000, partition=True)
    torch.cuda.synchronize()
    assert (out["cost"].cpu().numpy() == INF).all() and not out["partition"].cpu().numpy().any()
    hap.hap_problem_destroy(hp)
    bad = problems.tiny()
    bad.tff[0, 0, 0, 0, 0] = bad.tdf[0, 0, 0, 0, 0] * 2       # FFN slower than the layer that contains it
    with pytest.raises(hap.HapError) as e:
        hap.hap_problem_create(bad)
    assert e.value.name == "HAP_E_INVALID"
    hp2 = hap.hap_problem_create(problems.tiny())
    with pytest.raises(hap.HapError) as e:
        hap.hap_pipeline_dp(hp2, 0, 1)                          # before hap_enumerate
    assert e.value.name == "HAP_E_STATE"


@pytest.mark.parametrize("seed", range(8))
def test_random_small_problems_with_tight_memory(hap, seed):
    """Mixed layer kinds, recomputation policies, windows and tight capacities on small random problems;
    seeds >= 4 use three recomputation levels whose time factors are not multiples of 1024 (the general
    stage-cost formula) and policies that skip a level."""
    pb = problems.random_small(seed, N=9 + seed % 4, T=2 + seed % 2, nodes_per_type=((2, 2), (2, 1, 1))[seed % 2],
                               node_size=2, window=(seed % 2 == 0), first_dense=True)
    if seed >= 4:
        pb.xi_q = np.ascontiguousarray(np.array([1024, 512, 64], np.int32))
        pb.tau_q = np.ascontiguousarray(np.array([0, 300, 1000], np.int32))
        pb.rc_masks = np.ascontiguousarray(np.array([0b001, 0b011, 0b111, 0b101], np.uint32))
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    o = Oracle(pb)
    assert hp.n_cand == o.n_cand
    costs, bn, best, feas = o.search()
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs) and np.array_equal(out["bottleneck"].cpu().numpy(), bn)
    part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
    for idx in range(0, o.n_cand, 5):
        plan, _, _ = o.eval_index(idx)
        if plan["T_iter"] < INF:
            assert part[idx, :plan["PP"]].tolist() == plan["n"] and rec[idx, :plan["PP"]].tolist() == plan["r"]
    if best is not None:
        plan, _ = hap.hap_search_best(hp)
        assert plan["index"] == best["index"] and plan["n"] == best["n"] and plan["r"] == best["r"]
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("kw", [{}, {"window": True}])
def test_finite_cell_count_matches_stage_cost_enumeration(hap, kw):
    """hap_count_cells (the roofline's unit count) against a direct enumeration of (i, j, k) with the oracle's
    stage cost, candidate by candidate."""
    pb, hp, o = setup(hap, "tiny", **kw)
    n_rc = len(pb.rc_masks)
    for idx in list(range(0, o.n_cand, 37)) + [o.n_cand - 1]:
        p = o.find_pconf(idx)
        PP = int(o.pconfs["PP"][p])
        local = idx - int(o.pconfs["offset"][p])
        mp = o.decode(p, local // n_rc)
        rc = int(pb.rc_masks[local % n_rc])
        c2, _, coef, _ = o.layer_costs(p)
        want = 0
        for i in range(1, PP + 1):
            for j in range(i, pb.N - PP + i + 1):
                for k in range(i - 1, j):
                    want += o.stage_cost(p, mp, rc, c2, coef, i, k, j)[0] < INF
        assert hap.hap_count_cells(hp, idx, 1) == want, idx
    total = hap.hap_count_cells(hp, 0, hp.n_cand)
    assert total == sum(hap.hap_count_cells(hp, f, c) for f, c in ((0, 700), (700, hp.n_cand - 700)))


@pytest.mark.parametrize("name", CONFIGS)
def test_pruned_search_returns_the_same_plan(hap, name):
    """Lower-bound pruning against the running incumbent must not change the answer (strict bound, ties to the
    lowest index), whatever order the blocks ran in."""
    pb, hp, o = setup(hap, name)
    ref, stats0 = hap.hap_search_best(hp)
    hp2 = hap.hap_problem_create(pb, prune=1)
    hap.hap_enumerate(hp2)
    for _ in range(3):
        plan, stats = hap.hap_search_best(hp2)
        assert plan == ref
        assert stats["n_evaluated"] + stats["n_pruned"] == o.n_cand and stats0["n_pruned"] == 0
    if name in ("dsv2", "stress"):
        assert stats["n_pruned"] > 0
    # a sub-range that does not contain the global optimum
    first, count = o.n_cand // 3, o.n_cand // 5
    a, _ = hap.hap_search_range(hp, first, count)
    b, sb = hap.hap_search_range(hp2, first, count)
    assert a == b and sb["n_evaluated"] + sb["n_pruned"] == count
    hap.hap_problem_destroy(hp2)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}),
                                     ("dsv2", {}), ("stress", {})])
def test_fp64_mode_costs_within_1e9_relative(hap, name, kw):
    """fp64 mode: every candidate's iteration time and bottleneck within 1e-9 relative of the fp64 oracle,
    infeasible candidates identical, the chosen plan the oracle's (unless its two best costs are closer than
    1e-9 relative)."""
    pb, hp, o = setup(hap, name, **kw)
    out = hap.hap_pipeline_dp_f64(hp, 0, hp.n_cand, partition=True)
    torch.cuda.synchronize()
    got, gotb, part = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy(), out["partition"].cpu().numpy()
    done, costs, bn, parts = o.search_pconfs_f64(0, 1, threads=NTHREADS)
    assert done == o.n_cand
    fin = np.isfinite(costs)
    assert np.array_equal(fin, np.isfinite(got)) and np.array_equal(np.isfinite(bn), np.isfinite(gotb))
    assert (np.isposinf(got[~fin])).all()
    assert np.max(np.abs(got[fin] - costs[fin]) / costs[fin]) <= 1e-9
    bfin = np.isfinite(bn)
    assert np.max(np.abs(gotb[bfin] - bn[bfin]) / bn[bfin]) <= 1e-9
    # partitions: identical, except where two partitions tie at rounding level -- then the kernel's partition must
    # still be a partition of all N layers whose bottleneck and iteration time equal the oracle's within 1e-9 relative
    same = (part == parts).all(axis=1)
    assert not part[~fin].any()
    differ = np.nonzero(fin & ~same)[0]
    assert differ.size <= max(4, fin.sum() // 2000), differ.size
    for idx in differ:
        assert int(part[idx].sum()) == pb.N, idx
        assert abs(got[idx] - costs[idx]) <= 1e-9 * costs[idx] and abs(gotb[idx] - bn[idx]) <= 1e-9 * bn[idx], idx
    order = np.argsort(costs[fin], kind="stable")[:2]
    best_idx = np.nonzero(fin)[0][order]
    plan = hap.hap_search_range_f64(hp, 0, hp.n_cand)
    gap = (costs[best_idx[1]] - costs[best_idx[0]]) / costs[best_idx[0]] if len(best_idx) > 1 else 1.0
    assert plan["index"] == int(best_idx[0]) or gap <= 1e-9
    assert plan["T_iter_f64"] == pytest.approx(costs[plan["index"]], rel=1e-9)
    assert plan["n"] == parts[plan["index"], :plan["PP"]].tolist()
    # integer and fp64 modes pick plans of (nearly) the same cost
    iplan, _ = hap.hap_search_best(hp)
    assert abs(iplan["T_iter"] - plan["T_iter_f64"]) <= 1e-3 * plan["T_iter_f64"]


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}), ("dsv2", {})])
def test_refinement_pass_bit_exact(hap, name, kw):
    """HAP_OPT_REFINE: smallest stage-cost sum among the bottleneck-optimal partitions, against the oracle's
    refined evaluation of every candidate; plan and pruned plan included."""
    pb = problems.make_problem(name, **kw)
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs_refined(0, 1, threads=NTHREADS)
    for prune in (0, 1):
        hp = hap.hap_problem_create(pb, prune=prune, flags=hap.OPT_REFINE)
        hap.hap_enumerate(hp)
        if prune == 0:
            out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
            torch.cuda.synchronize()
            assert np.array_equal(out["cost"].cpu().numpy(), costs)
            assert np.array_equal(out["bottleneck"].cpu().numpy(), bn)
            part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
            for idx in range(0, o.n_cand, max(1, o.n_cand // 400)):
                ref = o.eval_index_refined(idx)
                if ref["T_iter"] < INF:
                    assert part[idx, :ref["PP"]].tolist() == ref["n"] and rec[idx, :ref["PP"]].tolist() == ref["r"], idx
            with pytest.raises(hap.HapError):
                hap.hap_pipeline_dp_f64(hp, 0, 1)
        plan, stats = hap.hap_search_best(hp)
        assert (plan["T_iter"], plan["index"]) == (bc, bi)
        ref = o.eval_index_refined(bi)
        assert plan["n"] == ref["n"] and plan["r"] == ref["r"] and plan["T_pipe"] == ref["T_pipe"]
        hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("seed", [4, 5])
def test_refinement_on_random_problems_with_general_levels(hap, seed):
    pb = problems.random_small(seed, N=9 + seed % 4, T=2 + seed % 2, nodes_per_type=((2, 2), (2, 1, 1))[seed % 2],
                               node_size=2, window=(seed % 2 == 0), first_dense=True)
    pb.xi_q = np.ascontiguousarray(np.array([1024, 512, 64], np.int32))
    pb.tau_q = np.ascontiguousarray(np.array([0, 300, 1000], np.int32))
    pb.rc_masks = np.ascontiguousarray(np.array([0b001, 0b011, 0b111, 0b101], np.uint32))
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs_refined(0, 1, threads=NTHREADS)
    hp = hap.hap_problem_create(pb, flags=hap.OPT_REFINE)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs)
    plan, _ = hap.hap_search_best(hp)
    assert (plan["T_iter"], plan["index"]) == (bc, bi)
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}), ("stress", {})])
def test_joint_device_state_recurrence(hap, name, kw):
    """hap_joint_bottleneck: equal to the oracle's joint recurrence on sampled configurations; equal to the minimum
    of the per-candidate bottlenecks wherever all sequences are enumerated; never above it for block orderings."""
    pb, hp, o = setup(hap, name, **kw)
    n_rc = len(pb.rc_masks)
    jb = hap.hap_joint_bottleneck(hp).cpu().numpy()
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    bn = out["bottleneck"].cpu().numpy()
    m = [0] * pb.T
    for t in pb.node_type:
        m[t] += int(pb.node_size[t])
    n_multiset = n_block_homog = 0
    for p in range(o.n_pconf):
        off, nmap, mode, G = (int(o.pconfs[f][p]) for f in ("offset", "nmap", "mode", "G"))
        homog = all(x % G == 0 for x in m)
        for rc in range(n_rc):
            enumerated = bn[off + rc: off + nmap * n_rc: n_rc].min()
            if not homog:
                assert jb[p, rc] == -1
            elif mode == 0:
                assert jb[p, rc] == enumerated, (p, rc)
                n_multiset += 1
            else:
                assert jb[p, rc] <= enumerated, (p, rc)       # block orderings are a subset of all sequences
                n_block_homog += 1
    assert n_multiset > 0
    if name == "stress":
        assert n_block_homog > 0
    rng = np.random.default_rng(1)
    small_pp = [p for p in range(o.n_pconf) if int(o.pconfs["PP"][p]) <= (8 if pb.N <= 32 else 4)]
    for p in rng.choice(small_pp, size=min(12, len(small_pp)), replace=False):
        for rc in range(n_rc):
            assert jb[p, rc] == o.joint_bottleneck(int(p), int(pb.rc_masks[rc])), (p, rc)


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {})])
def test_exact_pipeline_term_mode_bit_exact(hap, name, kw):
    """HAP_OPT_EXACT: the partition minimising sum + (M-1) max over all partitions of a candidate (limit sweep),
    against the oracle's sweep for every candidate; plan with and without pruning."""
    pb = problems.make_problem(name, **kw)
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs_exact(0, 1, threads=NTHREADS)
    for prune in (0, 1):
        hp = hap.hap_problem_create(pb, prune=prune, flags=hap.OPT_EXACT)
        hap.hap_enumerate(hp)
        if prune == 0:
            out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
            torch.cuda.synchronize()
            got = out["cost"].cpu().numpy()
            bad = np.nonzero(got != costs)[0]
            assert bad.size == 0, (bad[:5], got[bad[:5]], costs[bad[:5]])
            assert np.array_equal(out["bottleneck"].cpu().numpy(), bn)
            part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
            for idx in range(0, o.n_cand, max(1, o.n_cand // 300)):
                ex = o.eval_index_exact(idx)
                if ex["T_iter"] < INF:
                    assert part[idx, :ex["PP"]].tolist() == ex["n"] and rec[idx, :ex["PP"]].tolist() == ex["r"], idx
        plan, stats = hap.hap_search_best(hp)
        assert (plan["T_iter"], plan["index"]) == (bc, bi)
        hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("seed", [1, 4, 6])
def test_exact_mode_on_random_problems(hap, seed):
    pb = problems.random_small(seed, N=9 + seed % 4, T=2 + seed % 2, nodes_per_type=((2, 2), (2, 1, 1))[seed % 2],
                               node_size=2, window=(seed % 2 == 0), first_dense=True)
    if seed >= 4:
        pb.xi_q = np.ascontiguousarray(np.array([1024, 512, 64], np.int32))
        pb.tau_q = np.ascontiguousarray(np.array([0, 300, 1000], np.int32))
        pb.rc_masks = np.ascontiguousarray(np.array([0b001, 0b011, 0b111, 0b101], np.uint32))
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs_exact(0, 1, threads=NTHREADS)
    hp = hap.hap_problem_create(pb, flags=hap.OPT_EXACT)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs)
    for idx in range(0, o.n_cand, 41):
        ex = o.eval_index_exact(idx)
        if ex["T_iter"] < INF:
            assert ex["T_pipe"] == ex["brute_pipe"]
    hap.hap_problem_destroy(hp)


def _configs_sampled(o, stride):
    """Candidate index ranges of every `stride`-th configuration (what search_pconfs(0, stride) evaluates)."""
    n_rc = o.n_cand and len(o.pb.rc_masks)
    return [(int(o.pconfs["offset"][p]), int(o.pconfs["nmap"][p]) * n_rc) for p in range(0, o.n_pconf, stride)]


@pytest.mark.parametrize("mode,stride", [("refine", 5), ("exact", 23)])
def test_refinement_modes_on_the_stress_workload(hap, mode, stride):
    """The refinement and the exact pipeline term at the benchmark's size: every candidate of every `stride`-th
    configuration against the oracle; the bounded search (plain pass, per-candidate lower bounds, refinement only
    where the bound can still win) returns the minimum of the unbounded pass over all candidates."""
    pb = problems.stress()
    o = Oracle(pb)
    flag = hap.OPT_REFINE if mode == "refine" else hap.OPT_EXACT
    search = o.search_pconfs_refined if mode == "refine" else o.search_pconfs_exact
    done, _, _, costs, bn = search(0, stride, threads=NTHREADS)
    hp = hap.hap_problem_create(pb, flags=flag)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    got, gotb = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy()
    n = 0
    for off, cnt in _configs_sampled(o, stride):
        assert np.array_equal(got[off:off + cnt], costs[off:off + cnt]), off
        assert np.array_equal(gotb[off:off + cnt], bn[off:off + cnt]), off
        n += cnt
    assert n == done and (costs[costs >= 0] < INF).any()
    plan, stats = hap.hap_search_best(hp)
    am = int(np.argmin(got))
    assert (plan["T_iter"], plan["index"]) == (int(got[am]), am)
    # candidates without a feasible partition count as evaluated; nearly all others are cut by their bound
    assert stats["n_evaluated"] + stats["n_pruned"] == hp.n_cand and stats["n_pruned"] > 0.9 * int((got < INF).sum())
    # a range that does not hold the global optimum, and pruning by the configuration-level bound on top
    first, count = hp.n_cand // 4, hp.n_cand // 3
    sub, _ = hap.hap_search_range(hp, first, count)
    am = int(np.argmin(got[first:first + count]))
    assert (sub["T_iter"], sub["index"]) == (int(got[first + am]), first + am)
    hap.hap_problem_destroy(hp)
    hp = hap.hap_problem_create(pb, prune=1, flags=flag)
    hap.hap_enumerate(hp)
    assert hap.hap_search_best(hp)[0] == plan
    hap.hap_problem_destroy(hp)
