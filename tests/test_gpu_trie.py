"""The prefix-tree form of the pipeline recurrence (trie_dp_kernel) against the oracle and against
the one-warp-per-candidate kernel (HAP_OPT_NO_TRIE), through the C ABI.  Integer work: bit-exact."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from gen import problems  # noqa: E402
from oracle import Oracle, INF  # noqa: E402

NTHREADS = max(1, len(os.sched_getaffinity(0)))


@pytest.fixture(scope="module")
def hap():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    return hap


def _pass(hap, pb, flags, first=0, count=None, partition=True):
    hp = hap.hap_problem_create(pb, flags=flags)
    hap.hap_enumerate(hp)
    if count is None:
        count = hp.n_cand - first
    out = hap.hap_pipeline_dp(hp, first, count, partition=partition)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items() if v is not None}
    return hp, res


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiny", {"window": True}), ("small", {}), ("mixtral", {}), ("dsv2", {}), ("stress", {})])
def test_both_kernels_agree_on_every_candidate(hap, name, kw):
    """Costs, bottlenecks, partitions and recomputation levels of the whole candidate space."""
    pb = problems.make_problem(name, **kw)
    hp_t, tree = _pass(hap, pb, 0)
    hp_w, warp = _pass(hap, pb, hap.OPT_NO_TRIE)
    for key in ("cost", "bottleneck", "partition", "recompute"):
        bad = np.nonzero((tree[key] != warp[key]).reshape(len(tree[key]), -1).any(axis=1))[0]
        assert bad.size == 0, (key, bad[:8])
    # and the oracle on a sample (the full comparison with the oracle runs in test_gpu_parity)
    o = Oracle(pb)
    rng = np.random.default_rng(11)
    for idx in rng.integers(0, o.n_cand, 200).tolist():
        plan, _, _ = o.eval_index(idx)
        assert tree["cost"][idx] == plan["T_iter"] and tree["bottleneck"][idx] == plan["bottleneck"], idx
        if plan["T_iter"] < INF:
            PP = plan["PP"]
            assert tree["partition"][idx, :PP].tolist() == plan["n"] and tree["recompute"][idx, :PP].tolist() == plan["r"], idx
            assert not tree["partition"][idx, PP:].any()
        else:
            assert not tree["partition"][idx].any() and not tree["recompute"][idx].any()
    # searches, with and without pruning, return the same plan
    plan_t, st_t = hap.hap_search_best(hp_t)
    plan_w, st_w = hap.hap_search_best(hp_w)
    assert plan_t == plan_w
    assert st_t["n_evaluated"] == st_w["n_evaluated"] == o.n_cand and st_t["n_feasible"] == st_w["n_feasible"]
    am = int(np.argmin(tree["cost"]))
    assert plan_t["index"] == am and plan_t["T_iter"] == int(tree["cost"][am])
    hap.hap_problem_destroy(hp_t)
    hap.hap_problem_destroy(hp_w)
    hp_p = hap.hap_problem_create(pb, prune=1)
    hap.hap_enumerate(hp_p)
    plan_p, st_p = hap.hap_search_best(hp_p)
    assert plan_p == plan_t and st_p["n_evaluated"] + st_p["n_pruned"] == o.n_cand
    hap.hap_problem_destroy(hp_p)


def test_ragged_ranges_across_configurations(hap):
    """Ranges that start and end inside a configuration's candidates; everything outside stays untouched."""
    pb = problems.small()
    o = Oracle(pb)
    costs, bn, best, feas = o.search(0, o.n_cand)
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    rng = np.random.default_rng(5)
    for first, count in [(0, 2), (1, 7), (o.n_cand - 3, 3)] + [(int(a), int(b)) for a, b in zip(rng.integers(0, o.n_cand - 5000, 6), rng.integers(2, 5000, 6))]:
        out = hap.hap_pipeline_dp(hp, first, count, partition=True)
        torch.cuda.synchronize()
        assert np.array_equal(out["cost"].cpu().numpy(), costs[first:first + count]), (first, count)
        assert np.array_equal(out["bottleneck"].cpu().numpy(), bn[first:first + count]), (first, count)
        sub = costs[first:first + count]
        if sub.min() >= INF:
            with pytest.raises(hap.HapError) as e:
                hap.hap_search_range(hp, first, count)
            assert e.value.name == "HAP_E_INFEASIBLE"
            continue
        plan, stats = hap.hap_search_range(hp, first, count)
        assert plan["T_iter"] == int(sub.min()) and plan["index"] == first + int(np.argmin(sub))
        assert stats["n_evaluated"] == count
        want = o.eval_index(plan["index"])[0]          # the plan the winning block left, term by term
        for key in ("n", "r", "mask", "bottleneck", "T_pipe", "T_sync", "T_opt"):
            assert plan[key] == want[key], (first, count, key)
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("seed", range(6))
def test_random_problems_with_tight_memory_and_windows(hap, seed):
    """Small random problems (several types, tight capacities, general recomputation levels where the
    level-combined rows exist) against the oracle, every candidate."""
    pb = problems.random_small(20 + seed, N=8 + seed % 5, T=2 + seed % 2, nodes_per_type=((2, 2), (2, 1, 1))[seed % 2],
                               node_size=2, window=(seed % 3 != 0), first_dense=(seed % 2 == 0))
    if seed >= 3:       # three levels whose time factors are multiples of 1024, policies that skip a level
        pb.xi_q = np.ascontiguousarray(np.array([1024, 512, 64], np.int32))
        pb.tau_q = np.ascontiguousarray(np.array([0, 1024, 2048], np.int32))
        pb.rc_masks = np.ascontiguousarray(np.array([0b001, 0b011, 0b111, 0b101], np.uint32))
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=NTHREADS, want_costs=True)
    hp, tree = _pass(hap, pb, 0)
    assert np.array_equal(tree["cost"], costs) and np.array_equal(tree["bottleneck"], bn)
    for idx in range(0, o.n_cand, max(1, o.n_cand // 200)):
        plan, _, _ = o.eval_index(idx)
        if plan["T_iter"] < INF:
            assert tree["partition"][idx, :plan["PP"]].tolist() == plan["n"] and tree["recompute"][idx, :plan["PP"]].tolist() == plan["r"], idx
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("name,eta_q", [("tiny", 16), ("small", 24)])
def test_heterogeneous_communication_rule_in_the_tree_kernel(hap, name, eta_q):
    pb = problems.make_problem(name)
    pb.eta_q = eta_q
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=NTHREADS, want_costs=True)
    hp, tree = _pass(hap, pb, 0)
    assert np.array_equal(tree["cost"], costs) and np.array_equal(tree["bottleneck"], bn)
    assert (costs >= INF).sum() > (bn >= INF).sum()          # the rule dropped some candidates with a feasible partition
    hap.hap_problem_destroy(hp)


def test_large_multiset_class(hap):
    """12 870 distinct stage-type sequences per configuration (PP = 16 on the two-type cluster with no cap on the
    enumeration): the tree is cut into parts or, where it does not fit, the class runs one warp per candidate;
    either way the values are those of the oracle."""
    pb = problems.mixtral()
    pb.map_cap = 1 << 40
    pb.pp_list = np.ascontiguousarray(np.array([16], np.int32))
    pb.tp_list = pb.tp_list[:2]; pb.cp_list = pb.cp_list[:1]; pb.ep_list = pb.ep_list[:2]; pb.tpe_list = pb.tpe_list[:1]
    pb.mb_list = pb.mb_list[:2]
    for f in ("tdf", "tdb", "tff", "tfb"):
        setattr(pb, f, np.ascontiguousarray(getattr(pb, f)[:, :2, :1, :2]))
    pb.tpre = np.ascontiguousarray(pb.tpre[:, :2, :1, :2]); pb.tpost = np.ascontiguousarray(pb.tpost[:, :2, :1, :2])
    pb.rho = pb.rho[:2].copy()
    o = Oracle(pb)
    assert int(o.pconfs["nmap"][0]) == 12870
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=NTHREADS, want_costs=True)
    hp, tree = _pass(hap, pb, 0)
    assert np.array_equal(tree["cost"], costs) and np.array_equal(tree["bottleneck"], bn)
    rng = np.random.default_rng(2)
    for idx in rng.integers(0, o.n_cand, 100).tolist():
        plan, _, _ = o.eval_index(idx)
        if plan["T_iter"] < INF:
            assert tree["partition"][idx, :16].tolist() == plan["n"] and tree["recompute"][idx, :16].tolist() == plan["r"], idx
    plan, stats = hap.hap_search_best(hp)
    assert (plan["T_iter"], plan["index"]) == (bc, bi)
    hap.hap_problem_destroy(hp)


def test_many_random_problems_agree_between_the_two_kernels(hap):
    """Differential test without the oracle in the loop: a hundred random problems (two to four device types, window on
    and off, one to three recomputation levels, several policies, dense first layer or not, uniform-split ablation,
    heterogeneous-communication rule) through both kernels; every output must be identical."""
    shapes = [((2, 2), 2), ((2, 1, 1), 3), ((1, 1, 1, 1), 4), ((4, 2, 2), 3), ((3, 1), 2)]
    n_checked = 0
    for seed in range(100):
        nodes, T = shapes[seed % len(shapes)]
        pb = problems.random_small(100 + seed, N=6 + (seed * 7) % 19, T=T, nodes_per_type=nodes, node_size=2,
                                   window=(seed % 3 != 1), first_dense=(seed % 4 == 0))
        if seed % 5 == 2:
            pb.xi_q = np.ascontiguousarray(np.array([1024, 512, 64], np.int32))
            pb.tau_q = np.ascontiguousarray(np.array([0, 1024, 3072], np.int32))
            pb.rc_masks = np.ascontiguousarray(np.array([0b001, 0b011, 0b111, 0b101, 0b100], np.uint32))
        if seed % 5 == 3:
            pb.rc_masks = np.ascontiguousarray(np.array([0b01], np.uint32))
        if seed % 7 == 6:
            pb.uniform = 1
        if seed % 6 == 5:
            pb.eta_q = 40
        if seed % 8 == 7:
            pb.map_cap = 4                                  # forces block orderings with mixed stages
        hp_t, tree = _pass(hap, pb, 0)
        hp_w, warp = _pass(hap, pb, hap.OPT_NO_TRIE)
        for key in ("cost", "bottleneck", "partition", "recompute"):
            assert np.array_equal(tree[key], warp[key]), (seed, key)
        if (tree["cost"] < INF).any():
            assert hap.hap_search_best(hp_t)[0] == hap.hap_search_best(hp_w)[0], seed
        n_checked += len(tree["cost"])
        hap.hap_problem_destroy(hp_t)
        hap.hap_problem_destroy(hp_w)
    assert n_checked > 50000


@pytest.mark.parametrize("name", ["tiny", "small", "dsv2"])
def test_fp64_mode_agrees_between_the_two_kernels(hap, name):
    """fp64 mode: the tree kernel and the one-warp-per-candidate kernel follow the same steps up to the order of a
    few additions (stage constants, the sum over the stages of a plan); feasibility agrees exactly, costs and
    bottlenecks to rounding, partitions except where two splits tie to the last bits."""
    pb = problems.make_problem(name)
    res = {}
    for flags in (0, hap.OPT_NO_TRIE):
        hp = hap.hap_problem_create(pb, flags=flags)
        hap.hap_enumerate(hp)
        out = hap.hap_pipeline_dp_f64(hp, 0, hp.n_cand, partition=True)
        torch.cuda.synchronize()
        res[flags] = {k: v.cpu().numpy() for k, v in out.items()}
        hap.hap_problem_destroy(hp)
    a, b = res[0], res[hap.OPT_NO_TRIE]
    fin = np.isfinite(a["cost"])
    assert np.array_equal(fin, np.isfinite(b["cost"])) and fin.any()
    assert np.allclose(a["bottleneck"][fin], b["bottleneck"][fin], rtol=1e-13, atol=0.0)
    same_part = (a["partition"] == b["partition"]).all(axis=1)
    assert same_part[fin].mean() > 0.999
    both = fin & same_part
    assert np.allclose(a["cost"][both], b["cost"][both], rtol=1e-13, atol=0.0)
    assert np.array_equal(a["recompute"][both], b["recompute"][both])


@pytest.mark.parametrize("name", ["tiny", "small", "dsv2", "stress"])
def test_layer_costs_computed_inside_the_tree_blocks_equal_the_separate_launch(hap, name):
    """By default the blocks of the tree kernel compute Eq. 2 for their configuration themselves; HAP_OPT_NO_FUSE keeps
    the separate layer-cost launch.  Same arithmetic, so every output is identical, in both value types, and so are
    the searches (with pruning: the lower bound then comes from the block's own layer times)."""
    pb = problems.make_problem(name)
    hp_f, fused = _pass(hap, pb, 0)
    hp_s, sep = _pass(hap, pb, hap.OPT_NO_FUSE)
    for key in ("cost", "bottleneck", "partition", "recompute"):
        assert np.array_equal(fused[key], sep[key]), key
    out_f = hap.hap_pipeline_dp_f64(hp_f, 0, hp_f.n_cand)
    out_s = hap.hap_pipeline_dp_f64(hp_s, 0, hp_s.n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(out_f["cost"].cpu().numpy(), out_s["cost"].cpu().numpy())
    assert hap.hap_search_best(hp_f)[0] == hap.hap_search_best(hp_s)[0]
    assert hap.hap_launches_per_pass(hp_f) + 1 == hap.hap_launches_per_pass(hp_s)
    hap.hap_problem_destroy(hp_f)
    hap.hap_problem_destroy(hp_s)
    plans = []
    for flags in (0, hap.OPT_NO_FUSE):
        hp = hap.hap_problem_create(pb, prune=1, flags=flags)
        hap.hap_enumerate(hp)
        plan, stats = hap.hap_search_best(hp)
        assert stats["n_evaluated"] + stats["n_pruned"] == hp.n_cand
        plans.append(plan)
        if name in ("small", "dsv2"):
            plan64 = hap.hap_search_range_f64(hp, 0, hp.n_cand)
            assert plan64["index"] == plan["index"] and plan64["n"] == plan["n"]
        hap.hap_problem_destroy(hp)
    assert plans[0] == plans[1]
