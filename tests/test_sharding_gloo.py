"""Host-side multi-rank logic on CPU: work-balanced candidate ranges and the (cost, index) exchange
over torch.distributed (gloo, world size 2).  The per-rank minima come from the CPU oracle here,
because no GPU is present; the exchange and the sharding code are the ones bench.py uses."""
import os
import socket

import numpy as np
import pytest

from gen import problems
from oracle import Oracle
from paper_2609_39350_b200.sharding import (shard_ranges, combine_minima, exchange_minimum, exchange_minimum_tensor,
                                            recurrence_cells, NO_CANDIDATE)


def test_recurrence_cell_count_matches_the_loop_nest():
    """Cells of the plain recurrence that can hold a finite value: the first stage starts at k = 0,
    the last stage ends at j = N, every other stage tries each k in [i-1, j-1]."""
    for N, PP in ((16, 1), (16, 2), (16, 8), (96, 8), (96, 32), (7, 7)):
        cells = 0
        for i in range(1, PP + 1):
            for j in range(i, N - PP + i + 1):
                if PP == 1:
                    cells += 1 if j == N else 0
                elif i == 1:
                    cells += 1
                elif i == PP:
                    cells += (j - (i - 1)) if j == N else 0
                else:
                    cells += j - (i - 1)
        assert recurrence_cells(N, PP) == cells


@pytest.mark.parametrize("name", ["tiny", "small", "stress"])
@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_shards_are_contiguous_cover_everything_and_balance_work(name, world):
    pb = problems.make_problem(name)
    o = Oracle(pb)
    n_rc = len(pb.rc_masks)
    ranges = shard_ranges(o.pconfs, n_rc, pb.N, world)
    assert len(ranges) == world and ranges[0][0] == 0
    for (f0, c0), (f1, _) in zip(ranges, ranges[1:]):
        assert f0 + c0 == f1
    assert ranges[-1][0] + ranges[-1][1] == o.n_cand
    # work per shard within 25 % of the mean (per-candidate work is constant inside a configuration)
    per = np.repeat(np.array([recurrence_cells(pb.N, int(pp)) + 256.0 for pp in o.pconfs["PP"]]),
                    o.pconfs["nmap"].astype(np.int64) * n_rc)
    work = [per[f:f + c].sum() for f, c in ranges]
    if world <= 3 or name != "tiny":
        assert max(work) <= 1.25 * (sum(work) / world) + per.max()


def test_combine_minima_breaks_ties_by_index():
    assert combine_minima([(5, 9), (5, 3), (7, 0)]) == (5, 3)
    assert combine_minima([(1 << 62, 2 ** 64 - 1), (10, 4)]) == (10, 4)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, name, q, ranges):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        pb = problems.make_problem(name)
        o = Oracle(pb)
        first, count = (ranges or shard_ranges(o.pconfs, len(pb.rc_masks), pb.N, world))[rank]
        best = o.search(first, count)[2] if count else None
        mine = (best["T_iter"], best["index"]) if best is not None else NO_CANDIDATE
        # the tensor form takes the index relative to the range start, as hap_argmin returns it
        local = torch.tensor([mine[0], mine[1] - first if best is not None else mine[1]], dtype=torch.int64)
        combined_t = exchange_minimum_tensor(local, first if best is not None else 0)
        q.put((rank, mine, exchange_minimum(mine[0], mine[1]), tuple(int(x) for x in combined_t.tolist())))
    finally:
        dist.destroy_process_group()


def _run_ranks(name, world, ranges=None):
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, name, q, ranges)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=300) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    return got


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_two_rank_search_over_gloo_equals_the_single_rank_search(name):
    got = _run_ranks(name, 2)
    o = Oracle(problems.make_problem(name))
    _, _, best, _ = o.search()
    for rank, mine, combined, combined_t in got:
        assert combined == combined_t == (best["T_iter"], best["index"]), (rank, mine, combined, combined_t)
    assert len({m for _, m, _, _ in got}) == 2            # the two ranks really searched different ranges


@pytest.mark.parametrize("world", [3, 8])
def test_more_ranks_and_an_empty_shard(world):
    """World sizes 3 and 8 on the Tiny space; the last rank gets an empty range and contributes "no candidate"."""
    pb = problems.tiny()
    o = Oracle(pb)
    ranges = shard_ranges(o.pconfs, len(pb.rc_masks), pb.N, world - 1) + [(o.n_cand, 0)]
    assert sum(c for _, c in ranges) == o.n_cand
    got = _run_ranks("tiny", world, ranges)
    _, _, best, _ = o.search()
    for rank, mine, combined, combined_t in got:
        assert combined == combined_t == (best["T_iter"], best["index"]), (rank, mine, combined, combined_t)
    assert [m for r, m, _, _ in got if r == world - 1] == [NO_CANDIDATE]


def test_all_shards_empty_or_infeasible_yield_no_candidate():
    import torch
    t = exchange_minimum_tensor(torch.tensor(list(NO_CANDIDATE), dtype=torch.int64), 0)
    assert tuple(int(x) for x in t.tolist()) == NO_CANDIDATE
