"""The CUDA path on the hand-computed examples of tests/golden: its results are compared with the numbers derived
by hand there (not with the oracle), so a mistake that the oracle and the kernels shared would still show.

e8: Eq. 4's gradient-synchronisation and optimizer terms, each decided by a different stage than the bottleneck.
e9: a stage whose device group spans two device types (per-layer slowest member, smallest member's memory,
    slowest member's share in the load-balance window).
e10: Pruning 3 with the dispatch / combine traffic of stages that span device types."""
import json
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from hand_examples import e8_problem, e9_problem, e10_problem  # noqa: E402

GOLD = os.path.join(os.path.dirname(__file__), "golden")
INF = 1 << 62


def gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)["expect"]


@pytest.fixture(scope="module")
def hap():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    return hap


CASES = [(e8_problem, "e8_sync_opt_assembly.json", ("ABC", "BAC")), (e9_problem, "e9_mixed_type_stage.json", ("AB", "BA"))]


@pytest.mark.parametrize("make, gname, names", CASES)
@pytest.mark.parametrize("flags", [0, 16, 2, 4, 1])     # default, no prefix tree, refinement, exact sweep, no mapping table
def test_hand_values_of_the_candidates(hap, make, gname, names, flags):
    g = gold(gname)
    hp = hap.hap_problem_create(make(), flags=flags)
    n_pconf, n_cand = hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, n_cand, partition=True)
    torch.cuda.synchronize()
    cost, bott = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy()
    part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
    for name in names:
        want = g[name]
        i, PP = want["map_idx"], len(want["n"])
        assert int(cost[i]) == want["T_iter"] and int(bott[i]) == want["bottleneck"], (name, int(cost[i]))
        assert part[i, :PP].tolist() == want["n"]
        assert rec[i, :PP].tolist() == want.get("r", [0] * PP)
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("make, gname, names", CASES)
def test_hand_values_of_the_plan_terms(hap, make, gname, names):
    """hap_search_range on one candidate returns the plan with T_pipe, T_sync and T_opt separately."""
    g = gold(gname)
    for prune in (0, 1):
        hp = hap.hap_problem_create(make(), prune=prune)
        hap.hap_enumerate(hp)
        for name in names:
            want = g[name]
            plan, _ = hap.hap_search_range(hp, want["map_idx"], 1)
            for key in ("n", "bottleneck", "T_pipe", "T_sync", "T_opt", "T_iter"):
                assert plan[key] == want[key], (name, key, plan[key])
            if "masks" in g:
                assert plan["mask"] == g["masks"][name]
        if "best_index" in g:
            plan, _ = hap.hap_search_best(hp)
            assert plan["index"] == g["best_index"]
        hap.hap_problem_destroy(hp)


def test_hand_values_of_the_coefficients(hap):
    g = gold("e8_sync_opt_assembly.json")["coef"]
    hp = hap.hap_problem_create(e8_problem())
    hap.hap_enumerate(hp)
    c2, coef = hap.hap_eval_layer_costs(hp)
    torch.cuda.synchronize()
    coef = coef.cpu().numpy()[0]
    SLAT, SBW, OPT, CROSS = 8, 9, 11, 4
    for h, name in enumerate("ABC"):
        assert coef[h, SBW:SBW + 2].tolist() == g["sbw"][name] and coef[h, OPT:OPT + 2].tolist() == g["opt"][name]
        assert coef[h, SLAT] == g["slat"] and coef[h, CROSS:CROSS + 3].tolist() == [g["kp2p_cross"]] * 3
    hap.hap_problem_destroy(hp)
    m = gold("e9_mixed_type_stage.json")["mem_coef"]
    hp = hap.hap_problem_create(e9_problem())
    hap.hap_enumerate(hp)
    _, coef = hap.hap_eval_layer_costs(hp)
    torch.cuda.synchronize()
    row = coef.cpu().numpy()[0, 0]
    assert [row[13 + 1], row[15 + 1], row[17], row[18], row[19]] == [m["mw"], m["ma"], m["mx"], m["mpre"], m["mpre"]]
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("make, gname, names", CASES)
def test_fp64_mode_tracks_the_hand_values(hap, make, gname, names):
    g = gold(gname)
    hp = hap.hap_problem_create(make())
    n_pconf, n_cand = hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp_f64(hp, 0, n_cand, partition=True)
    torch.cuda.synchronize()
    cost, part = out["cost"].cpu().numpy(), out["partition"].cpu().numpy()
    for name in names:
        want = g[name]
        PP = len(want["n"])
        assert abs(cost[want["map_idx"]] - want["T_iter"]) <= PP + 8        # unrounded coefficients: < 1 ns per term
        assert part[want["map_idx"], :PP].tolist() == want["n"]
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("flags", [0, 16, 2, 4, 1])     # default, no prefix tree, refinement, exact sweep, no mapping table
def test_hand_values_of_the_wider_heterogeneous_communication_rule(hap, flags):
    g = gold("e10_hetero_dispatch.json")
    cases = [(k, v, 1) for k, v in g["pruned"].items()] + [(k, v, 0) for k, v in g["pruned_without_option"].items()]
    for eta_q, want, option in cases:
        pb = e10_problem()
        pb.eta_q, pb.het_coll = int(eta_q), option
        hp = hap.hap_problem_create(pb, flags=flags)
        n_pconf, n_cand = hap.hap_enumerate(hp)
        assert (n_pconf, n_cand) == (1, 2)
        out = hap.hap_pipeline_dp(hp, 0, n_cand, partition=True)
        torch.cuda.synchronize()
        cost, bott = out["cost"].cpu().numpy(), out["bottleneck"].cpu().numpy()
        for name, dropped in zip(("AB", "BA"), want):
            i = g[name]["map_idx"]
            assert int(bott[i]) == g[name]["bottleneck"]
            assert int(cost[i]) == (INF if dropped else g[name]["T_iter"]), (eta_q, name, int(cost[i]))
        if not all(want):
            plan, stats = hap.hap_search_best(hp)
            assert plan["index"] == (1 if not want[1] else 0) and stats["n_feasible"] == want.count(False)
        if flags == 0:
            fo = hap.hap_pipeline_dp_f64(hp, 0, n_cand)
            torch.cuda.synchronize()
            assert [not np.isfinite(x) for x in fo["cost"].cpu().numpy()] == want
        hap.hap_problem_destroy(hp)


def test_hand_values_of_the_cross_type_dispatch_coefficient(hap):
    g = gold("e10_hetero_dispatch.json")
    hp = hap.hap_problem_create(e10_problem())
    hap.hap_enumerate(hp)
    c2, coef = hap.hap_eval_layer_costs(hp)
    c2f, coeff = hap.hap_eval_layer_costs_f64(hp)
    torch.cuda.synchronize()
    assert coef.cpu().numpy()[0, :, hap.COEF["KXD"]].tolist() == g["kxd"]
    assert np.allclose(coeff.cpu().numpy()[0, :, hap.COEF["KXD"]], g["kxd_f64"], rtol=1e-14, atol=0)
    assert c2.cpu().numpy()[0].sum(axis=2).tolist() == [g["layer_sum"]["A"], g["layer_sum"]["B"]]
    hap.hap_problem_destroy(hp)
