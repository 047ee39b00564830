"""GPU parity of the vocabulary-sharded verify step against the CPU oracle.

Only one GPU is assumed: the ranks' column slices all sit on it and their kernels are ordinary launches of one
stream, issued rank after rank; the all-reduce between launches is replaced by combining the ranks' exchange
buffers in rank order.  What is checked is what a real job must get: every rank ends with exactly the outputs
the oracle computes from the full rows (accept/reject decisions, paths, winning root, new token).
"""
import dataclasses

import numpy as np
import pytest
import torch

from mcsd_inputs import gammas, parent_array, verify_inputs, workload
from oracle import mcsd_oracle as orc
from tests.helpers import condition_uniforms, to_np

pytestmark = pytest.mark.gpu

KEYS = ("accept_len", "out_tokens", "out_nodes", "best_root")


@pytest.fixture(scope="module")
def m():
    from paper_2409_10644_b200 import build
    build.build()
    import paper_2409_10644_b200 as pkg
    return pkg


def _sharded_case(m, w, worlds, parent=None, B=None, V=None, gamma="workload", tweak=None, step=0, bounds=None):
    from paper_2409_10644_b200 import dist as mdist
    parent = parent_array(w.n_roots, w.branching) if parent is None else parent
    vin = verify_inputs(w, step, "cuda", parent=parent, B=B, V=V)
    B, N, V = vin["p"].shape
    if isinstance(gamma, str):
        gamma = None if w.gamma is None else gammas(dataclasses.replace(w, B=B), step)
    if tweak is not None:
        tweak(vin)
    host = {k: to_np(v) for k, v in vin.items()}
    ua, ub = condition_uniforms(host["p"], host["q"], host["tokens"], parent, gamma, host["u_accept"], host["u_bonus"])
    ref = orc.verify_tree(host["p"], host["q"], host["tokens"], parent, gamma, ua, ub)
    tm = m.mcsd_build_mask(parent)
    dev = vin["p"].device
    g_d = None if gamma is None else torch.from_numpy(np.asarray(gamma, dtype=np.int32)).to(dev)
    ua_d, ub_d = torch.from_numpy(ua).to(dev), torch.from_numpy(ub).to(dev)
    k = mdist.max_children(parent)
    for world in worlds:
        if bounds is not None:
            cuts = bounds
            world = len(cuts) - 1
        else:
            cuts = [mdist.vocab_shard_range(V, r, world)[0] for r in range(world)] + [V]
        shards = []
        for r in range(world):
            v0, v1 = cuts[r], cuts[r + 1]
            assert v1 > v0
            shards.append(m.VocabShard(vin["p"][:, :, v0:v1].contiguous(), vin["q"][:, :, v0:v1].contiguous(), v0, V,
                                       r, world, vin["tokens"], tm, g_d, ua_d, ub_d))
        outs = mdist.drive_vocab_shards(shards, mdist.reduce_on_one_device, k)
        torch.cuda.synchronize()
        for r, got in enumerate(outs):                     # every rank holds the full result
            for key in KEYS:
                assert np.array_equal(got[key].cpu().numpy(), ref[key]), (world, r, key)
        del shards, outs
    return ref


def test_sharded_verify_tiny_workload(m):
    _sharded_case(m, workload(1), worlds=(1, 2, 3, 4, 8))


def test_sharded_verify_llama_shapes(m):
    _sharded_case(m, workload(2), worlds=(2, 8))
    ref = _sharded_case(m, workload(4), worlds=(1, 2, 4))
    assert ref["accept_len"].max() > 0


def test_sharded_verify_sliced_tree_and_forest(m):
    _sharded_case(m, workload(3), worlds=(2, 3))
    w5 = dataclasses.replace(workload(5), B=8)
    ref = _sharded_case(m, w5, worlds=(2, 4))
    assert len(set(ref["best_root"].tolist())) > 1
    # fork of 16 chains: up to 16 rejections at one node, 17 rounds
    _sharded_case(m, workload(7), worlds=(2,), B=4)
    torch.cuda.empty_cache()


def test_sharded_verify_edge_cases(m):
    w = workload(1)
    # column ranges of odd width and odd start take the scalar-load path; a one-column rank
    _sharded_case(m, w, worlds=(0,), B=3, V=1001, bounds=[0, 1, 334, 335, 1001])
    _sharded_case(m, w, worlds=(3,), B=3, V=13)
    # gamma = 0: nothing is tested; one-node tree
    ref = _sharded_case(m, w, worlds=(2,), B=2, gamma=np.array([0, 2]))
    assert ref["accept_len"][0] == 0
    _sharded_case(m, w, worlds=(2,), parent=np.array([-1], dtype=np.int32), B=2)
    # draft equal to target: every first candidate accepted, no residual pass at all
    def same(vin):
        vin["q"].copy_(vin["p"])
    ref = _sharded_case(m, w, worlds=(2, 4), B=2, tweak=same)
    assert list(ref["accept_len"]) == [3, 3]
    # draft mass on a token the target never emits: all rejected, residual equals the target row; the whole
    # mass of the draft sits in the first rank's columns
    def disjoint(vin):
        vin["p"][:, :, 0] = 0.0
        vin["p"].div_(vin["p"].sum(-1, keepdim=True))
        vin["q"].zero_()
        vin["q"][:, :, 0] = 1.0
        vin["tokens"][:, 1:] = 0
    ref = _sharded_case(m, w, worlds=(2, 4), B=2, tweak=disjoint)
    assert list(ref["accept_len"]) == [0, 0]
    # target mass confined to the last rank's columns: the ranks before it report zero mass
    def tail_only(vin):
        V = vin["p"].shape[-1]
        vin["p"][:, :, : V - V // 4] = 0.0
        vin["p"].div_(vin["p"].sum(-1, keepdim=True))
    _sharded_case(m, w, worlds=(4,), B=2, tweak=tail_only)


def test_sharded_verify_equals_the_single_gpu_entry_point(m):
    # same inputs through mcsd_verify_tree and through four column slices: identical integer outputs
    from paper_2409_10644_b200 import dist as mdist
    w = workload(3)
    parent = parent_array(w.n_roots, w.branching)
    vin = verify_inputs(w, 2, "cuda", parent=parent)
    B, N, V = vin["p"].shape
    gamma = gammas(w, 2)
    host = {k: to_np(v) for k, v in vin.items()}
    ua, ub = condition_uniforms(host["p"], host["q"], host["tokens"], parent, gamma, host["u_accept"], host["u_bonus"])
    tm = m.mcsd_build_mask(parent)
    dev = vin["p"].device
    g_d = torch.from_numpy(np.asarray(gamma, dtype=np.int32)).to(dev)
    ua_d, ub_d = torch.from_numpy(ua).to(dev), torch.from_numpy(ub).to(dev)
    one = m.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, g_d, ua_d, ub_d)
    shards = []
    for r in range(4):
        v0, v1 = mdist.vocab_shard_range(V, r, 4)
        shards.append(m.VocabShard(vin["p"][:, :, v0:v1].contiguous(), vin["q"][:, :, v0:v1].contiguous(), v0, V, r, 4,
                                   vin["tokens"], tm, g_d, ua_d, ub_d))
    outs = mdist.drive_vocab_shards(shards, mdist.reduce_on_one_device, mdist.max_children(parent))
    torch.cuda.synchronize()
    for key in KEYS:
        assert torch.equal(outs[0][key], one[key]), key


# ---------------------------------------------------------------------------------------------------------
# The real driver end to end: two processes, a process group, this library's kernels in each
# ---------------------------------------------------------------------------------------------------------
def _two_process_rank(rank, world, port, q, widx, B, V):
    """One rank of dist.verify_tree_vocab_sharded.  Both ranks use GPU 0 (one GPU is all there is): each launches its
    own kernels from its own process and the reductions between them go through a gloo group, so nothing on the device
    waits for the other rank."""
    import os
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    try:
        torch.cuda.set_device(0)
        dist.init_process_group("gloo", rank=rank, world_size=world)
        import paper_2409_10644_b200 as m
        from paper_2409_10644_b200 import dist as mdist
        w = workload(widx)
        parent = parent_array(w.n_roots, w.branching)
        vin = verify_inputs(w, 0, "cuda", parent=parent, B=B, V=V)          # same seeds: both ranks draw the same rows
        gamma = None if w.gamma is None else gammas(dataclasses.replace(w, B=B), 0)
        host = {k: to_np(v) for k, v in vin.items()}
        ua, ub = condition_uniforms(host["p"], host["q"], host["tokens"], parent, gamma, host["u_accept"], host["u_bonus"])
        ref = orc.verify_tree(host["p"], host["q"], host["tokens"], parent, gamma, ua, ub)
        tm = m.mcsd_build_mask(parent)
        dev = vin["p"].device
        g_d = None if gamma is None else torch.from_numpy(np.asarray(gamma, dtype=np.int32)).to(dev)
        v0, v1 = mdist.vocab_shard_range(V, rank, world)
        out = mdist.verify_tree_vocab_sharded(vin["p"][:, :, v0:v1].contiguous(), vin["q"][:, :, v0:v1].contiguous(), v0, V,
                                              vin["tokens"], tm, g_d, torch.from_numpy(ua).to(dev), torch.from_numpy(ub).to(dev))
        torch.cuda.synchronize()
        bad = [k for k in KEYS if not np.array_equal(out[k].cpu().numpy(), ref[k])]
        q.put((rank, bad, int(ref["accept_len"].sum())))
        dist.barrier()
        dist.destroy_process_group()
    except Exception as e:                                       # report instead of leaving the parent waiting
        q.put((rank, ["exception: %r" % (e,)], -1))
        raise


@pytest.mark.parametrize("widx,B,V", [(2, 3, 1000), (5, 4, 777)])
def test_vocab_sharded_driver_with_two_processes_and_a_process_group(m, widx, B, V):
    import socket
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_two_process_rank, args=(r, 2, port, q, widx, B, V)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=300) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1]
    for rank, bad, total in got:
        assert bad == [], (rank, bad)                            # every rank ends with the oracle's integers
    assert got[0][2] == got[1][2] and got[0][2] >= 0
