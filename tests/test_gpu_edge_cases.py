"""Edge cases of the CUDA path against the oracle: maximum sizes, degenerate sizes, one device type,
many recomputation levels and policies, in-kernel unranking instead of the mapping table, value limits."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from gen import problems  # noqa: E402
from gen.problems import DENSE, MOE  # noqa: E402
from oracle import Oracle, INF  # noqa: E402


@pytest.fixture(scope="module")
def hap():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    assert torch.cuda.is_available()
    return hap


def full_compare(hap, pb, tables_every=0, flags=0):
    hp = hap.hap_problem_create(pb, flags=flags)
    hap.hap_enumerate(hp)
    o = Oracle(pb)
    assert (hp.n_pconf, hp.n_cand) == (o.n_pconf, o.n_cand)
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=8, want_costs=True)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs)
    assert np.array_equal(out["bottleneck"].cpu().numpy(), bn)
    part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
    step = max(1, o.n_cand // 300)
    for idx in range(0, o.n_cand, step):
        plan, _, _ = o.eval_index(idx)
        if plan["T_iter"] < INF:
            assert part[idx, :plan["PP"]].tolist() == plan["n"] and rec[idx, :plan["PP"]].tolist() == plan["r"], idx
    if tables_every:
        for idx in range(0, o.n_cand, tables_every):
            t = hap.hap_pipeline_dp(hp, idx, 1, tables=True)
            torch.cuda.synchronize()
            plan, edp, ech = o.eval_index(idx, tables=True)
            assert np.array_equal(t["dp_table"].cpu().numpy()[0, :plan["PP"] + 1], edp), idx
            assert np.array_equal(t["choice"].cpu().numpy()[0, :plan["PP"] + 1], ech), idx
    if (costs < INF).any():
        plan, stats = hap.hap_search_best(hp)
        assert (plan["T_iter"], plan["index"]) == (bc, bi)
    hap.hap_problem_destroy(hp)
    return o, costs


def _model_problem(N, pp_list, nodes_per_type, node_size, P_tf, **kw):
    T = len(P_tf)
    kind = kw.pop("kind", [MOE] * N)
    pb = problems._build("edge", kw.pop("seed", 11), N=N, S=2048, H=1024, E=8, k=2, n_shared=0, F_dense=4096,
                         F_exp=2048, nq=8, nkv=8, V=32000, GB=kw.pop("GB", 64), kind=kind, P_tf=P_tf,
                         C_gb=kw.pop("C_gb", [80, 64, 48, 40][:T]), node_size=[node_size] * T,
                         bw_intra=[900.0, 600.0, 400.0, 300.0][:T], node_type=problems._nodes(list(nodes_per_type)),
                         bw_inter_fixed=50.0, bw_inter_random=False, zipf_alpha=1.2, mb_list=kw.pop("mb_list", [1]),
                         rc_masks=kw.pop("rc_masks", [0b11]), delta_q=kw.pop("delta_q", 205),
                         map_cap=kw.pop("map_cap", 2048))
    pb.pp_list = np.ascontiguousarray(np.array(pp_list, np.int32))
    for k, v in kw.items():
        setattr(pb, k, v)
    return pb


def test_maximum_layers_and_stages(hap):
    """N = 255 layers, PP up to 32, four device types; multiset and block-mode classes."""
    pb = _model_problem(255, [1, 2, 4, 8, 16, 32], (1, 1, 1, 1), 8, [400, 300, 250, 150], map_cap=4096,
                        kind=[DENSE] * 3 + [MOE] * 252)
    pb.tp_list = pb.tp_list[:1]; pb.tpe_list = pb.tpe_list[:1]; pb.cp_list = pb.cp_list[:1]; pb.ep_list = pb.ep_list[:2]
    for f in ("tdf", "tdb", "tff", "tfb"):
        setattr(pb, f, np.ascontiguousarray(getattr(pb, f)[:, :1, :1]))
    pb.tpre = np.ascontiguousarray(pb.tpre[:, :1, :1]); pb.tpost = np.ascontiguousarray(pb.tpost[:, :1, :1])
    pb.rho = pb.rho[:2].copy()
    pb.cap_eff[:] = pb.cap_eff // 4            # make recomputation and infeasibility occur
    o, costs = full_compare(hap, pb, tables_every=997)
    assert set(o.pconfs["PP"].tolist()) == {1, 2, 4, 8, 16, 32} and 0 < (costs < INF).sum() < o.n_cand
    pb.delta_q = -1                             # the same without the window: full-width bands, longer spans
    pb.pp_list = np.ascontiguousarray(np.array([1, 4, 32], np.int32))
    full_compare(hap, pb, tables_every=71)


@pytest.mark.parametrize("N,pp", [(1, [1]), (2, [1, 2]), (8, [8]), (5, [1, 4])])
def test_degenerate_layer_counts(hap, N, pp):
    """One layer; as many stages as layers (every stage holds exactly one layer)."""
    W = max(pp)
    pb = _model_problem(N, pp, (W // 2 or 1, W - (W // 2 or 1)) if W > 1 else (1,), 1,
                        [400, 200] if W > 1 else [400], delta_q=-1, GB=8)
    full_compare(hap, pb, tables_every=1)


def test_single_device_type_and_window(hap):
    pb = _model_problem(24, [1, 2, 4, 8], (2,), 4, [300], rc_masks=[0b01, 0b11], mb_list=[1, 2])
    o, costs = full_compare(hap, pb, tables_every=13)
    assert set(o.pconfs["nmap"].tolist()) == {1}       # one type: exactly one mapping per configuration


def test_four_recompute_levels_eight_policies(hap):
    pb = _model_problem(20, [2, 4], (2, 1, 1), 4, [400, 300, 200], C_gb=[12, 9, 6], delta_q=-1, mb_list=[1, 4])
    pb.xi_q = np.ascontiguousarray(np.array([1024, 700, 300, 40], np.int32))
    pb.tau_q = np.ascontiguousarray(np.array([0, 256, 640, 1024], np.int32))
    pb.rc_masks = np.ascontiguousarray(np.array([1, 2, 4, 8, 3, 5, 10, 15], np.uint32))
    pb.cap_eff[:] = pb.cap_eff // 3
    o, costs = full_compare(hap, pb, tables_every=101)
    levels = set()
    for idx in range(0, o.n_cand, 11):
        if costs[idx] < INF:
            levels |= set(o.eval_index(idx)[0]["r"])
    assert levels == {0, 1, 2, 3}


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_in_kernel_unranking_without_the_mapping_table(hap, name):
    full_compare(hap, problems.make_problem(name), flags=hap.OPT_NO_MAPTAB)


def test_value_limits_are_reported(hap):
    pb = problems.tiny()
    big = pb.copy()
    for f in ("tdf", "tdb"):
        getattr(big, f)[:] = getattr(big, f) * 1.0e5 + 1.0e11       # layers of > 2^36 ns
    hp = hap.hap_problem_create(big)
    hap.hap_enumerate(hp)
    with pytest.raises(hap.HapError) as e:
        hap.hap_search_best(hp)
    assert e.value.name == "HAP_E_RANGE"
    hap.hap_problem_destroy(hp)
    huge_batch = pb.copy(GB=1 << 19)                                # 2^19 sequences x 16 layers > 2^22
    with pytest.raises(hap.HapError) as e:
        hap.hap_problem_create(huge_batch)
    assert e.value.name == "HAP_E_RANGE"


# flags: default, one warp per candidate, refinement, exact sweep (the refinement modes on one threshold per workload)
@pytest.mark.parametrize("name,eta_q,flags", [(n, e, f) for n, e in (("tiny", 2048), ("tiny", 128), ("small", 2048), ("small", 24), ("mixtral", 512))
                                              for f in (0, 16, 2, 4) if f < 2 or n == "tiny" or e == 2048])
def test_heterogeneous_communication_pruning_with_dispatch_of_mixed_stages(hap, name, eta_q, flags):
    """The wider reading of Pruning 3: the dispatch and combine traffic of stages that span device types counts as
    cross-type communication, so candidates are dropped that the narrow reading keeps (already at the paper's eta = 2)."""
    pb = problems.make_problem(name)
    pb.eta_q = eta_q
    o_narrow = Oracle(pb)
    narrow = {0: o_narrow.search_pconfs, 16: o_narrow.search_pconfs, 2: o_narrow.search_pconfs_refined,
              4: o_narrow.search_pconfs_exact}[flags](0, 1, threads=8, want_costs=True)[3]
    pb.het_coll = 1
    o = Oracle(pb)
    search = {0: o.search_pconfs, 16: o.search_pconfs, 2: o.search_pconfs_refined, 4: o.search_pconfs_exact}[flags]
    done, bc, bi, costs, bn = search(0, 1, threads=8, want_costs=True)
    assert ((costs >= INF) & (narrow < INF)).sum() > 0 and not ((costs < INF) & (narrow >= INF)).any()
    hp = hap.hap_problem_create(pb, flags=flags)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs) and np.array_equal(out["bottleneck"].cpu().numpy(), bn)
    for prune in (0, 1):
        hq = hap.hap_problem_create(pb, flags=flags, prune=prune)
        hap.hap_enumerate(hq)
        plan, stats = hap.hap_search_best(hq)
        assert (plan["T_iter"], plan["index"]) == (bc, bi)
        hap.hap_problem_destroy(hq)
    if flags == 0:
        got = hap.hap_pipeline_dp_f64(hp, 0, hp.n_cand)["cost"].cpu().numpy()
        cf = o.search_pconfs_f64(0, 1, threads=8)[1]
        assert (np.isfinite(got) == np.isfinite(cf)).mean() > 0.9999       # a candidate exactly at the threshold may fall either way
        fin = np.isfinite(got) & np.isfinite(cf)
        assert np.max(np.abs(got[fin] - cf[fin]) / cf[fin]) <= 1e-9
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("name,eta_q", [("tiny", 64), ("tiny", 16), ("small", 2048), ("small", 24), ("mixtral", 12)])
def test_heterogeneous_communication_pruning(hap, name, eta_q):
    """Pruning 3: candidates whose cross-type transfer time exceeds eta x the mean stage time cost +INF."""
    pb = problems.make_problem(name)
    base = Oracle(pb).search_pconfs(0, 1, threads=8, want_costs=True)[3]
    pb.eta_q = eta_q
    o, costs = full_compare(hap, pb)
    dropped = int(((costs >= INF) & (base < INF)).sum())
    assert (dropped > 0) == (eta_q < 2048)
    assert np.array_equal(costs[costs < INF], base[costs < INF])
    # fp64 mode applies the same rule to the unrounded values
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp_f64(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    done, cf, bf, parts = o.search_pconfs_f64(0, 1, threads=8)
    got = out["cost"].cpu().numpy()
    agree = np.isfinite(got) == np.isfinite(cf)
    assert agree.mean() > 0.9999                      # a candidate exactly at the threshold may fall either way
    fin = np.isfinite(got) & np.isfinite(cf)
    assert np.max(np.abs(got[fin] - cf[fin]) / cf[fin]) <= 1e-9
    hap.hap_problem_destroy(hp)


@pytest.mark.parametrize("name", ["tiny", "small", "mixtral"])
def test_uniform_partition_ablation(hap, name):
    """HAP_OPT_UNIFORM (the paper's "non-uniform partitioning disabled" ablation): stages take floor/ceil(N/PP)
    layers.  Parity with the oracle; the uniform optimum can never beat the non-uniform one when the window is off."""
    pb = problems.make_problem(name)
    pb.uniform = 1
    o, costs = full_compare(hap, pb, tables_every=997)
    for idx in range(0, o.n_cand, max(1, o.n_cand // 50)):
        plan, _, _ = o.eval_index(idx)
        if plan["T_iter"] < INF:
            assert max(plan["n"]) - min(plan["n"]) <= 1
    free = problems.make_problem(name)
    free.delta_q = -1
    best_free = Oracle(free).search_pconfs(0, 1, threads=8)[1]
    assert costs.min() >= best_free
    # the joint recurrence honours the same restriction
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    jb = hap.hap_joint_bottleneck(hp).cpu().numpy()
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    bn = out["bottleneck"].cpu().numpy()
    n_rc = len(pb.rc_masks)
    for p in range(o.n_pconf):
        if int(o.pconfs["mode"][p]) == 0:
            off, nmap = int(o.pconfs["offset"][p]), int(o.pconfs["nmap"][p])
            for rc in range(n_rc):
                assert jb[p, rc] == bn[off + rc: off + nmap * n_rc: n_rc].min()
    hap.hap_problem_destroy(hp)


def test_device_memory_of_destroyed_problems_is_reused(hap):
    """Problems created one after another (different sizes in between) give the oracle's plan every time: a
    recycled, dirty arena must not leak anything of its previous owner into the next problem; releasing the
    cache returns the memory to the driver."""
    torch.cuda.synchronize()
    hap.hap_release_cached_memory()
    expected = {}
    for name in ("small", "tiny", "small", "mixtral", "small", "tiny"):
        pb = problems.make_problem(name)
        if name not in expected:
            o = Oracle(pb)
            done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=8, want_costs=True)
            expected[name] = (bc, bi, costs)
        bc, bi, costs = expected[name]
        hp = hap.hap_problem_create(pb)
        hap.hap_enumerate(hp)
        plan, stats = hap.hap_search_best(hp)
        assert (plan["T_iter"], plan["index"]) == (bc, bi), name
        out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
        torch.cuda.synchronize()
        assert np.array_equal(out["cost"].cpu().numpy(), costs), name
        hap.hap_problem_destroy(hp)
    free_cached, _ = torch.cuda.mem_get_info()
    hap.hap_release_cached_memory()
    free_released, _ = torch.cuda.mem_get_info()
    assert free_released > free_cached           # idle blocks went back to the driver
    hap.hap_release_cached_memory()              # nothing left: a no-op


@pytest.mark.parametrize("make", [lambda: problems.tiny(), lambda: problems.with_link_efficiency_table(problems.small(), seed=3),
                                  lambda: problems.random_small(23, N=12, T=3, nodes_per_type=(2, 1, 1), node_size=2, window=True, first_dense=True)])
def test_saved_problem_loads_into_an_identical_one(hap, make):
    """hap_problem_save / hap_problem_load: the blob carries every input; the loaded problem enumerates the same
    space and gives the same costs and plan.  Damaged blobs are refused."""
    pb = make()
    hp = hap.hap_problem_create(pb)
    blob = hap.hap_problem_save(hp)
    hap.hap_enumerate(hp)
    ref = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    plan, _ = hap.hap_search_best(hp)
    assert hap.hap_problem_save(hp) == blob                       # saving is repeatable and independent of the state
    hp2 = hap.hap_problem_load(blob)
    assert (hp2.N, hp2.T, hp2.n_rc) == (hp.N, hp.T, hp.n_rc)
    assert hap.hap_enumerate(hp2) == (hp.n_pconf, hp.n_cand)
    out = hap.hap_pipeline_dp(hp2, 0, hp2.n_cand, partition=True)
    plan2, _ = hap.hap_search_best(hp2)
    torch.cuda.synchronize()
    for key in ("cost", "bottleneck", "partition", "recompute"):
        assert torch.equal(out[key], ref[key]), key
    assert plan2 == plan
    assert hap.hap_problem_save(hp2) == blob
    hap.hap_problem_destroy(hp)
    hap.hap_problem_destroy(hp2)
    for bad in (blob[:-1], blob[:40], b"", blob + b"\0", b"X" + blob[1:], blob[:8] + (len(blob) + 8).to_bytes(8, "little") + blob[16:]):
        with pytest.raises(hap.HapError) as e:
            hap.hap_problem_load(bad)
        assert e.value.name == "HAP_E_INVALID"
    # a length field inside the blob that points past its end
    cut = bytearray(blob)
    cut[16 + 64 + 0:16 + 64 + 8] = (1 << 40).to_bytes(8, "little")
    with pytest.raises(hap.HapError):
        hap.hap_problem_load(bytes(cut))


def test_enumeration_and_trees_reused_across_problems_of_the_process(hap):
    """Problems on the same cluster with different profiled tables share the cached enumeration and prefix trees;
    a problem that differs in anything the trees depend on (capacities order, window, compute rates) must not.
    Every variant is checked against the oracle, in one process, interleaved."""
    base = problems.small()
    variants = []
    faster = base.copy()
    faster.tdf *= 0.7; faster.tdb *= 0.7; faster.tff *= 0.7; faster.tfb *= 0.7            # new tables, same cluster
    variants.append(faster)
    caps = base.copy()
    caps.cap_eff = np.ascontiguousarray(base.cap_eff[::-1].copy())                         # another type binds the memory
    variants.append(caps)
    win = base.copy()
    win.delta_q = 100                                                                      # narrower window
    variants.append(win)
    rates = base.copy()
    rates.P = np.ascontiguousarray(base.P[::-1].copy())                                    # other window shares
    variants.append(rates)
    for pb in [base] + variants + [base, faster]:
        hp = hap.hap_problem_create(pb)
        hap.hap_enumerate(hp)
        o = Oracle(pb)
        assert (hp.n_pconf, hp.n_cand) == (o.n_pconf, o.n_cand)
        out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
        torch.cuda.synchronize()
        done, costs, bn, parts, levels = o.search_pconfs_plans(0, 1, threads=max(1, len(os.sched_getaffinity(0))))
        assert np.array_equal(out["cost"].cpu().numpy(), costs)
        assert np.array_equal(out["partition"].cpu().numpy(), parts) and np.array_equal(out["recompute"].cpu().numpy(), levels)
        hap.hap_problem_destroy(hp)
