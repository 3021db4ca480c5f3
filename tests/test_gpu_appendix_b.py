"""Appendix B's iteration latency of the plans the dynamic program chose (hap_eval_appendix_b) against the
oracle's plain evaluation of the same expression, through the C ABI.  Integer work: bit-exact."""
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


@pytest.mark.parametrize("name,kw,sample", [("tiny", {}, 0), ("tiny", {"window": True}, 0), ("small", {}, 1500),
                                            ("mixtral", {}, 1500), ("dsv2", {}, 800), ("stress", {}, 800)])
def test_appendix_b_latency_of_the_chosen_plans(hap, name, kw, sample):
    pb = problems.make_problem(name, **kw)
    o = Oracle(pb)
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    res = hap.hap_eval_appendix_b(hp, 0, hp.n_cand, out["partition"], out["recompute"], detail=True)
    torch.cuda.synchronize()
    cost = out["cost"].cpu().numpy()
    t_b, det = res["t_iter"].cpu().numpy(), res["detail"].cpu().numpy()
    part, rec = out["partition"].cpu().numpy(), out["recompute"].cpu().numpy()
    # infeasible candidates (no partition) stay infeasible; the appendix's value never exceeds the closed form when
    # the steady-state multiplier is not clipped
    assert np.array_equal(t_b >= INF, cost >= INF)
    idxs = range(o.n_cand) if not sample else np.random.default_rng(8).integers(0, o.n_cand, sample).tolist()
    n_rc = len(pb.rc_masks)
    cache = {}
    checked = 0
    for idx in idxs:
        if cost[idx] >= INF:
            continue
        p = o.find_pconf(int(idx))
        if p not in cache:
            c2, _, coef, _ = o.layer_costs(p)
            cache = {p: (c2, coef)}
        c2, coef = cache[p]
        PP = int(o.pconfs["PP"][p])
        mp = o.decode(p, (int(idx) - int(o.pconfs["offset"][p])) // n_rc)
        r = o.appendix_b(p, mp, c2, coef, part[idx, :PP].tolist(), rec[idx, :PP].tolist())
        assert (int(t_b[idx]), int(det[idx, 0]), int(det[idx, 1]), int(det[idx, 2])) == (r.T_iter, r.T_edge, r.T_middle, r.s_max), idx
        if int(o.pconfs["M"][p]) >= r.s_max + 1:
            assert t_b[idx] <= cost[idx]
        checked += 1
    assert checked > 0
    # sub-range with its own buffers, and a plan that does not cover the layers
    first, count = max(0, hp.n_cand // 3), min(257, hp.n_cand - hp.n_cand // 3)
    sub = hap.hap_eval_appendix_b(hp, first, count, out["partition"][first:first + count].contiguous(),
                                  out["recompute"][first:first + count].contiguous())
    bad_part = out["partition"][:4].clone()
    bad_part[:, 0] += 1
    bad = hap.hap_eval_appendix_b(hp, 0, 4, bad_part, out["recompute"][:4].contiguous())
    torch.cuda.synchronize()
    assert np.array_equal(sub["t_iter"].cpu().numpy(), t_b[first:first + count])
    assert (bad["t_iter"].cpu().numpy() >= INF).all()
    hap.hap_problem_destroy(hp)
