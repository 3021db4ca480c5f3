"""Inputs of the hand-computed examples that both the oracle pins and the CUDA parity tests use (data only:
the expected values live in tests/golden with their derivations)."""
import numpy as np

from gen import problems
from gen.problems import DENSE, MOE


def e8_problem():
    pb = problems.blank(N=6, S=2048, H=1024, E=4, k=2, GB=16, P_tf=[400, 200, 100], C_gb=[100000] * 3,
                        node_size=[4, 4, 4], nodes_per_type=[1, 1, 1], pp_list=(3,), kind=[DENSE] + [MOE] * 5,
                        F_dense=4096, F_exp=2048)
    fwd = {0: (3000000.0, 2000000.0), 1: (1500000.0, 1000000.0), 2: (1200000.0, 800000.0)}
    for h, (d, m) in fwd.items():
        row = np.array([d] + [m] * 5)
        pb.tdf[h, 0, 0, 0] = row
        pb.tdb[h, 0, 0, 0] = 2 * row
        pb.tff[h, 0, 0, 0] = row / 2
        pb.tfb[h, 0, 0, 0] = row
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.bw_intra[:] = [400.0, 100.0, 400.0]
    pb.node_bw_inter[:] = 25.0
    pb.chi, pb.ovl_dp = 0.7, 0.5
    pb.copt[:] = [0.012, 0.006, 0.048]
    return pb


def e9_problem():
    pb = problems.blank(N=8, S=1024, H=1024, E=4, k=2, GB=16, P_tf=[300, 100], C_gb=[100, 2], node_size=[6, 2],
                        nodes_per_type=[1, 1], pp_list=(2,), F_exp=1024, R=2)
    pb.tdf[0, 0, 0, 0] = 1000.0 * np.array([100, 300, 200, 400, 100, 300, 200, 400])
    pb.tdb[0, 0, 0, 0] = 1000.0 * np.array([500, 300, 600, 500, 500, 300, 600, 500])
    pb.tdf[1, 0, 0, 0] = 1000.0 * np.array([250, 200, 300, 100, 250, 200, 300, 100])
    pb.tdb[1, 0, 0, 0] = 1000.0 * np.array([400, 700, 500, 900, 400, 700, 500, 900])
    pb.tff[:] = pb.tdf / 2
    pb.tfb[:] = pb.tdb / 2
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.bw_intra[:] = 400.0
    pb.node_bw_inter[:] = 25.0
    pb.copt[:] = [0.01, 0.002]
    pb.act_coef[:] = [0.0, 1024.0]
    pb.delta_q = 205
    assert pb.cap_eff.tolist() == [100 << 30, 2 << 30]
    return pb


def e10_problem():
    pb = problems.blank(N=4, S=1024, H=1024, E=4, k=2, GB=16, P_tf=[300, 100], C_gb=[100000, 100000], node_size=[6, 2],
                        nodes_per_type=[1, 1], pp_list=(2,), ep_list=(2,), kind=[DENSE, MOE, MOE, MOE], F_exp=1024)
    for h, (d, m) in enumerate(((300000.0, 400000.0), (380000.0, 500000.0))):
        row = np.array([d, m, m, m])
        pb.tdf[h, 0, 0, 0] = row
        pb.tdb[h, 0, 0, 0] = 2 * row
        pb.tff[h, 0, 0, 0] = row / 2
        pb.tfb[h, 0, 0, 0] = row
    pb.alpha[:] = [2000.0, 8000.0, 12000.0]
    pb.bw_intra[:] = [400.0, 200.0]
    pb.node_bw_inter[:] = [25.0, 50.0]
    pb.chi, pb.gamma, pb.ovl_dp = 0.7, 0.5, 0.0
    pb.rho[:] = 1.5
    pb.het_coll = 1
    return pb
