"""The self-checking build of the library (-DHAP_CHECKED): the kernels compare the indices and shared-memory
addresses they form with their bounds before use and report violations through hap_self_check.  The same
problems as the parity tests run through it in a child process; results must equal the oracle's and no check
site may fire.  The normal build answers HAP_E_STATE."""
import json
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
import numpy as np, torch
sys.path.insert(0, sys.argv[1])
import paper_2609_39350_b200 as hap
from gen import problems
from oracle import Oracle, INF
report = {}
cases = [("tiny", problems.tiny()), ("tiny_window", problems.make_problem("tiny", window=True)), ("small", problems.small()),
         ("dsv2_like", problems.random_small(23, N=12, T=3, nodes_per_type=(2, 1, 1), node_size=2, window=True, first_dense=True)),
         ("random", problems.random_small(21, N=9, T=2, nodes_per_type=(2, 2), node_size=2, window=False, first_dense=False))]
for name, pb in cases:
    o = Oracle(pb)
    done, bc, bi, costs, bn = o.search_pconfs(0, 1, threads=4, want_costs=True)
    hp = hap.hap_problem_create(pb)
    hap.hap_enumerate(hp)
    out = hap.hap_pipeline_dp(hp, 0, hp.n_cand, partition=True)
    plan, stats = hap.hap_search_best(hp)
    sim = hap.hap_simulate_1f1b(hp, 0, hp.n_cand, out["partition"], out["recompute"])
    jb = hap.hap_joint_bottleneck(hp)
    torch.cuda.synchronize()
    report[name] = dict(costs_equal=bool(np.array_equal(out["cost"].cpu().numpy(), costs)),
                        bottlenecks_equal=bool(np.array_equal(out["bottleneck"].cpu().numpy(), bn)),
                        plan_equal=(plan["T_iter"], plan["index"]) == (bc, bi),
                        sites=hap.hap_self_check())
    hap.hap_problem_destroy(hp)
print("REPORT " + json.dumps(report))
"""


def test_checked_build_runs_the_parity_cases_without_a_violation():
    from paper_2609_39350_b200.build import build_library
    build_library(checked=True)
    assert torch.cuda.is_available()
    env = dict(os.environ, HAP_LIBRARY="checked")
    r = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [ln for ln in r.stdout.splitlines() if ln.startswith("REPORT ")][-1]
    report = json.loads(line[len("REPORT "):])
    assert len(report) == 5
    for name, rep in report.items():
        assert rep["costs_equal"] and rep["bottlenecks_equal"] and rep["plan_equal"], (name, rep)
        assert rep["sites"] == 0, (name, "check sites fired: " + bin(rep["sites"]))


def test_normal_build_has_no_checks():
    import paper_2609_39350_b200 as hap
    from paper_2609_39350_b200.build import build_library
    build_library()
    if os.environ.get("HAP_LIBRARY") == "checked":
        pytest.skip("the suite itself runs on the self-checking build")
    with pytest.raises(hap.HapError) as e:
        hap.hap_self_check()
    assert e.value.name == "HAP_E_STATE"
