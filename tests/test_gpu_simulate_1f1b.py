"""Event simulation of the 1F1B schedule for the plans the dynamic program chose (hap_simulate_1f1b) against the
oracle's plain simulation of the same schedule, through the C ABI.  Integer work: bit-exact."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from gen import problems  # noqa: E402
from oracle import Oracle, INF  # noqa: E402


@pytest.fixture(scope="module")
def hap():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    assert torch.cuda.is_available(), "the gpu tests need a CUDA device"
    return hap


@pytest.mark.parametrize("name,kw,sample", [("tiny", {}, 0), ("tiny", {"window": True}, 0), ("small", {}, 1200),
                                            ("mixtral", {}, 1200), ("dsv2", {}, 500), ("stress", {}, 500)])
def test_simulated_schedule_of_the_chosen_plans(hap, name, kw, sample):
    pb = problems.make_problem(name, **kw)
    o = Oracle(pb)
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    # the whole space for the small configs; for the large ones the sampled candidates, as one range each
    n_rc = len(pb.rc_masks)
    if not sample:
        out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
        res = hap.hap_simulate_1f1b(hp, 0, hp.n_cand, out["partition"], out["recompute"], detail=True)
        torch.cuda.synchronize()
        cost = out["cost"].cpu().numpy()
        t_s, det = res["t_iter"].cpu().numpy(), res["detail"].cpu().numpy()
        part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
        assert np.array_equal(t_s >= INF, cost >= INF)
        todo = [(i, cost[i], t_s[i], det[i], part[i], rec[i]) for i in range(o.n_cand)]
    else:
        todo = []
        for idx in np.random.default_rng(9).integers(0, o.n_cand, sample).tolist():
            first = max(0, int(idx) - 3)
            count = min(7, hp.n_cand - first)
            out = hap.hap_pipeline_dp(hp, first, count, partition=True)
            res = hap.hap_simulate_1f1b(hp, first, count, out["partition"], out["recompute"], detail=True)
            torch.cuda.synchronize()
            k = int(idx) - first
            todo.append((int(idx), int(out["cost"][k]), int(res["t_iter"][k]), res["detail"][k].cpu().numpy(),
                         out["partition"][k].cpu().numpy(), out["recompute"][k].cpu().numpy()))
    cache = {}
    checked = 0
    for idx, cst, ts, dt, pt, rc in todo:
        if cst >= INF:
            assert ts >= INF
            continue
        p = o.find_pconf(int(idx))
        if p not in cache:
            c2, _, coef, _ = o.layer_costs(p)
            cache = {p: (c2, coef)}
        c2, coef = cache[p]
        PP = int(o.pconfs["PP"][p])
        mp = o.decode(p, (int(idx) - int(o.pconfs["offset"][p])) // n_rc)
        r = o.simulate_1f1b(p, mp, c2, coef, pt[:PP].tolist(), rc[:PP].tolist())
        assert (int(ts), int(dt[0]), int(dt[1])) == (r.T_iter, r.T_pipe_sim, r.T_pipe_closed), idx
        # Eq. 4's iteration latency of the same plan is the closed pipeline term plus the same T_sync + T_opt
        assert int(cst) - int(dt[1]) == int(ts) - int(dt[0]) == r.T_sync + r.T_opt
        checked += 1
    assert checked > 0
    hap.hap_problem_destroy(hp)


def test_invalid_plans_sub_ranges_and_identical_stages(hap):
    pb = problems.tiny()
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    full = hap.hap_simulate_1f1b(hp, 0, hp.n_cand, out["partition"], out["recompute"])
    first, count = hp.n_cand // 3, min(257, hp.n_cand - hp.n_cand // 3)
    sub = hap.hap_simulate_1f1b(hp, first, count, out["partition"][first:first + count].contiguous(),
                                out["recompute"][first:first + count].contiguous())
    bad_part = out["partition"][:4].clone()
    bad_part[:, 0] += 1
    bad = hap.hap_simulate_1f1b(hp, 0, 4, bad_part, out["recompute"][:4].contiguous())
    torch.cuda.synchronize()
    assert np.array_equal(sub["t_iter"].cpu().numpy(), full["t_iter"].cpu().numpy()[first:first + count])
    assert (bad["t_iter"].cpu().numpy() >= INF).all()
    with pytest.raises(hap.HapError):
        hap.hap_simulate_1f1b(hp, hp.n_cand - 1, 2, out["partition"], out["recompute"])
    hap.hap_problem_destroy(hp)
    # identical stages on one device type with free transfers: the schedule takes exactly (M + PP - 1) c, Eq. 4's
    # pipeline term; many micro-batches (M = 512) exercise the ring of end times well past its length
    for N, PP, GB in ((12, 4, 8), (16, 8, 512), (32, 32, 64), (6, 1, 4)):
        pbu = problems.blank(N=N, S=1024, H=512, E=4, k=2, GB=GB, P_tf=[100], C_gb=[100000], node_size=[1],
                             nodes_per_type=[PP], pp_list=(PP,))
        pbu.tdf[:] = 5000.0; pbu.tdb[:] = 10000.0; pbu.tff[:] = 1000.0; pbu.tfb[:] = 2000.0
        pbu.bw_intra[:] = 1.0e15; pbu.node_bw_inter[:] = 1.0e15
        hpu = hap.hap_problem_create(pbu)
        hap.hap_enumerate(hpu)
        o = hap.hap_pipeline_dp(hpu, 0, 1, partition=True)
        s = hap.hap_simulate_1f1b(hpu, 0, 1, o["partition"], o["recompute"], detail=True)
        torch.cuda.synchronize()
        c = (N // PP) * 15000
        assert o["partition"][0, :PP].tolist() == [N // PP] * PP
        assert s["detail"][0].tolist() == [(GB + PP - 1) * c, (GB + PP - 1) * c]
        hap.hap_problem_destroy(hpu)
