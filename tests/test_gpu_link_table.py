"""The communication-primitive table (link efficiency by message size) through the C ABI: layer costs,
coefficients, every candidate and the plan against the oracle.  Integer mode bit-exact, fp64 identical."""
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


@pytest.mark.parametrize("name", ["tiny", "small", "mixtral", "dsv2"])
def test_costs_with_a_link_efficiency_table(hap, name):
    pb = problems.with_link_efficiency_table(problems.make_problem(name), seed=3)
    o = Oracle(pb)
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    c2, coef = hap.hap_eval_layer_costs(hp)
    c2f, coeff = hap.hap_eval_layer_costs_f64(hp)
    torch.cuda.synchronize()
    c2, coef, c2f, coeff = c2.cpu().numpy(), coef.cpu().numpy(), c2f.cpu().numpy(), coeff.cpu().numpy()
    for p in range(0, o.n_pconf, 1 if o.n_pconf <= 600 else 7):
        ec2, ec2f, ecoef, ecoeff = o.layer_costs(p)
        assert np.array_equal(c2[p], ec2) and np.array_equal(coef[p], ecoef), p
        assert np.array_equal(c2f[p], ec2f) and np.array_equal(coeff[p], ecoeff), p
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=NTHREADS, want_costs=True)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand)
    torch.cuda.synchronize()
    assert np.array_equal(out["cost"].cpu().numpy(), costs) and np.array_equal(out["bottleneck"].cpu().numpy(), bn)
    plan, _ = hap.hap_search_best(hp)
    assert (plan["T_iter"], plan["index"]) == (bc, bi)
    # the table changes the answer of the model (it is not a no-op on these inputs)
    base = Oracle(problems.make_problem(name)).search_pconfs(0, 1, threads=NTHREADS, want_costs=True)[3]
    assert (costs[costs < INF] != base[costs < INF]).any()
    hap.hap_problem_destroy(hp)


def test_bad_tables_are_rejected(hap):
    pb = problems.with_link_efficiency_table(problems.tiny())
    for change in ("descending", "zero_eff", "eff_above_one", "too_many"):
        bad = pb.copy()
        if change == "descending":
            bad.fsize = np.ascontiguousarray(bad.fsize[::-1])
        elif change == "zero_eff":
            bad.feff[1, 2] = 0.0
        elif change == "eff_above_one":
            bad.feff[2, 0] = 1.5
        else:
            bad.fsize = np.ascontiguousarray(np.arange(1, 18, dtype=np.float64) * 1e6)
            bad.feff = np.ascontiguousarray(np.full((3, 17), 0.5))
        with pytest.raises(hap.HapError) as e:
            hap.hap_problem_create(bad)
        assert e.value.name == "HAP_E_INVALID", change
