"""Host-side logic: gamma -> row count, batch sharding, and the two-rank (gloo) aggregation used for N > 1."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from mcsd_inputs import parent_array, workload
from oracle import mcsd_oracle as orc


@pytest.fixture(scope="module")
def m():
    from paper_2409_10644_b200 import build
    build.build()
    import paper_2409_10644_b200 as pkg
    return pkg


def test_n_active_from_gamma_matches_the_oracle_slice(m):
    for n_roots, br in [(1, (4, 2, 2, 1)), (8, (1, 2, 2, 1, 1, 1)), (1, (4, 2, 2, 1, 1, 1, 1, 1))]:
        parent = parent_array(n_roots, br)
        _, ls = orc.tree_levels(parent)
        gam = np.arange(0, len(br) + 1)
        got = m.n_active_from_gamma(ls, gam)
        assert list(got) == [orc.n_active_for_gamma(parent, int(g)) for g in gam]
    w = workload(5)
    _, ls = orc.tree_levels(parent_array(w.n_roots, w.branching))
    assert list(m.n_active_from_gamma(ls, [1, 2, 3, 4, 5, 6])) == [16, 32, 64, 96, 128, 160]


def test_shard_batch_partitions_every_batch(m):
    for B in (1, 2, 7, 16, 33):
        for ws in (1, 2, 3, 8):
            spans = [m.shard_batch(B, r, ws) for r in range(ws)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(spans[i][1] == spans[i + 1][0] for i in range(ws - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        m.shard_batch(4, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2409_10644_b200 import shard_batch
    from paper_2409_10644_b200.dist import aggregate
    rng = np.random.default_rng(5)
    B, V = 5, 13
    parent = parent_array(1, (2, 2))
    N = len(parent)
    x = rng.random((B, N, V)) + 1e-3
    p = x / x.sum(-1, keepdims=True)
    y = rng.random((B, N, V)) + 1e-3
    qq = y / y.sum(-1, keepdims=True)
    tokens = rng.integers(0, V, (B, N))
    ua, ub = rng.random((B, N)), rng.random((B, N))
    lo, hi = shard_batch(B, rank, world)
    # every rank verifies its own sequences and nothing is exchanged on the data path
    local = orc.verify_tree(p[lo:hi], qq[lo:hi], tokens[lo:hi], parent, None, ua[lo:hi], ub[lo:hi])
    units, ms = aggregate(units_local=float((hi - lo) * N), ms_local=10.0 * (rank + 1))
    gathered = [None] * world
    dist.all_gather_object(gathered, (lo, hi, local["accept_len"].tolist(), local["out_tokens"].tolist()))
    if rank == 0:
        full = orc.verify_tree(p, qq, tokens, parent, None, ua, ub)
        ok = True
        for (l, h, al, ot) in gathered:
            ok &= al == full["accept_len"][l:h].tolist() and ot == full["out_tokens"][l:h].tolist()
        q.put((ok, units, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_batch_sharding_over_gloo(m):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    ok, units, ms = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
    assert units == 5 * 7 and ms == 20.0      # units add up over ranks, time is the slowest rank's


def test_paper_shaped_workloads_and_early_stop_gammas():
    """Section 4.1: the static configuration (2; 4,3,1,1) has 82 nodes; the fork W = 16, D = 5 hangs 80 draft tokens
    off the last emitted token.  The early-stop stand-in gives reproducible draft lengths in 1..D that do vary."""
    from mcsd_inputs import gammas, parent_array, workload
    w6, w7 = workload("paper_static_2_4_3_1_1"), workload("paper_fork_w16_d5")
    assert w6.n_nodes == 2 + 2 * 40 and w6.n_roots == 2
    p7 = parent_array(w7.n_roots, w7.branching)
    assert len(p7) == 1 + 16 * 5 and int((p7 == 0).sum()) == 16
    for n in range(17, len(p7)):                      # every deeper node continues exactly one chain
        assert int((p7 == p7[n]).sum()) == 1
    assert list(gammas(w6)) == [4] * w6.B
    seen = set()
    for step in range(6):
        g = gammas(w7, step)
        assert np.array_equal(g, gammas(w7, step))
        assert g.min() >= 1 and g.max() <= 5
        seen |= set(g.tolist())
    assert len(seen) >= 3
