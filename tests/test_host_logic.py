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


# ----------------------------------------------------------------------------------------------
# vocabulary-sharded verify: column ranges, and the exchange protocol over two gloo ranks
# ----------------------------------------------------------------------------------------------

def test_vocab_shard_ranges_cover_the_vocabulary():
    from paper_2409_10644_b200.dist import max_children, vocab_shard_range
    for V in (33, 1000, 32000, 32001, 128256):
        for ws in (1, 2, 3, 8):
            spans = [vocab_shard_range(V, r, ws) for r in range(ws)]
            assert spans[0][0] == 0 and spans[-1][1] == V
            assert all(spans[i][1] == spans[i + 1][0] for i in range(ws - 1))
            assert all(lo % 4 == 0 and hi > lo for lo, hi in spans)
    with pytest.raises(ValueError):
        vocab_shard_range(13, 0, 5)          # four 4-id units cannot feed five ranks
    with pytest.raises(ValueError):
        vocab_shard_range(100, 2, 2)
    assert max_children(parent_array(1, (4, 2, 2, 1))) == 4
    assert max_children(parent_array(8, (1, 2, 2))) == 2
    assert max_children(np.array([-1])) == 0


class _CpuShard:
    """Test-side stand-in for one rank's kernels (numpy, fp64) with the interface the driver expects, so that the
    order of launches and reductions can be exercised over a CPU process group.  It restates what the four
    per-rank steps exchange; the product has no such path."""

    def __init__(self, p, q, v0, V_total, rank, world, tokens, parent, ua, ub):
        self.p, self.q, self.v0, self.V, self.rank, self.world = p, q, v0, V_total, rank, world
        self.tokens, self.parent, self.ua, self.ub = tokens, parent, ua, ub
        B, N, _ = p.shape
        self.B, self.N = B, N
        self.kids = [[c for c in range(N) if parent[c] == u] for u in range(N)]
        self.pq = torch.zeros((B, N, 2), dtype=torch.float64)
        self.y = torch.zeros((B, N), dtype=torch.float64)
        self.mass = torch.zeros((world, B, 2), dtype=torch.float64)
        nl = int(orc.tree_levels(parent)[0].max()) + 1
        self.nl = nl
        self.out = {"accept_len": torch.zeros(B, dtype=torch.int32), "out_tokens": torch.full((B, nl + 1), -1, dtype=torch.int32),
                    "out_nodes": torch.full((B, nl), -1, dtype=torch.int32), "best_root": torch.zeros(B, dtype=torch.int32)}

    def gather(self):
        self.pq.zero_()
        for b in range(self.B):
            for c in range(self.N):
                u, x = self.parent[c], int(self.tokens[b, c]) - self.v0
                if u >= 0 and 0 <= x < self.p.shape[2]:
                    self.pq[b, c, 0], self.pq[b, c, 1] = self.p[b, u, x], self.q[b, u, x]

    def round(self, r):
        if r == 0:
            self.stage = np.array([[0 if self.kids[u] else -1 for u in range(self.N)]] * self.B)
            self.pend = np.zeros((self.B, self.N), dtype=bool)
            self.c = np.zeros((self.B, self.N))
            self.Y = np.ones((self.B, self.N))
            self.next = -np.ones((self.B, self.N), dtype=int)
            self.stop_c = np.zeros((self.B, self.N))
        y_in = self.y.numpy().copy()
        self.y.zero_()
        for b in range(self.B):
            for u in range(self.N):
                if self.stage[b, u] < 0:
                    continue
                if self.pend[b, u]:
                    Y = y_in[b, u]
                    if not Y > 0:
                        self.c[b, u], Y = 0.0, 1.0
                    self.Y[b, u], self.pend[b, u] = Y, False
                    self.stage[b, u] += 1
                if self.stage[b, u] >= len(self.kids[u]):
                    self.stop_c[b, u], self.stage[b, u] = self.c[b, u], -1
                    continue
                child = self.kids[u][self.stage[b, u]]
                px, qx = float(self.pq[b, child, 0]), float(self.pq[b, child, 1])
                num = max(px - self.c[b, u] * qx, 0.0)
                acc = min(1.0, num / (self.Y[b, u] * qx)) if qx > 0 else (1.0 if num > 0 else 0.0)
                if self.ua[b, child] < acc:
                    self.next[b, u], self.stage[b, u] = child, -1
                else:
                    self.c[b, u] += self.Y[b, u]
                    self.pend[b, u] = True
                    self.y[b, u] = float(np.maximum(self.p[b, u] - self.c[b, u] * self.q[b, u], 0.0).sum())

    def _dist(self, b, u):
        return np.maximum(self.p[b, u] - self.stop_c[b, u] * self.q[b, u], 0.0)

    def select(self):
        self.mass.zero_()
        self.stop, self.slot = [], []
        roots = [n for n in range(self.N) if self.parent[n] < 0]
        for b in range(self.B):
            paths = []
            for r in roots:
                u, path = r, []
                while self.next[b, u] >= 0:
                    u = int(self.next[b, u])
                    path.append(u)
                paths.append(path)
            best = max(range(len(roots)), key=lambda i: (len(paths[i]), -i))
            toks = ([int(self.tokens[b, roots[best]])] if len(roots) > 1 else []) + [int(self.tokens[b, n]) for n in paths[best]]
            self.out["accept_len"][b], self.out["best_root"][b] = len(paths[best]), best
            self.out["out_tokens"][b] = -1
            self.out["out_nodes"][b] = -1
            self.out["out_tokens"][b, :len(toks)] = torch.tensor(toks, dtype=torch.int32)
            self.out["out_nodes"][b, :len(paths[best])] = torch.tensor(paths[best], dtype=torch.int32)
            u = paths[best][-1] if paths[best] else roots[best]
            self.stop.append(u)
            self.slot.append(len(toks))
            d = self._dist(b, u)
            pos = np.nonzero(d > 0)[0]
            self.mass[self.rank, b, 0] = float(d.sum())
            self.mass[self.rank, b, 1] = float(self.v0 + pos[-1] + 1) if pos.size else 0.0

    def pick(self):
        for b in range(self.B):
            u = self.stop[b]
            masses = self.mass[:, b, 0].numpy()
            target = float(self.ub[b, u]) * float(masses.sum())
            base, owner = 0.0, -1
            for r in range(self.world):
                if base + masses[r] > target:
                    owner = r
                    break
                base += masses[r]
            tok = -1
            if owner < 0:
                last = float(self.mass[:, b, 1].max())
                tok = int(last) - 1 if last > 0 else self.V - 1
            elif owner == self.rank:
                cs = base + np.cumsum(self._dist(b, u))
                tok = self.v0 + int(np.nonzero(cs > target)[0][0])
            self.out["out_tokens"][b, self.slot[b]] = tok


def _vocab_rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2409_10644_b200.dist import _all_reduce_group, drive_vocab_shards, max_children, vocab_shard_range
    rng = np.random.default_rng(11)
    B, V = 6, 40
    ok = True
    for parent in (parent_array(1, (3, 2)), parent_array(2, (2, 1, 1))):
        N = len(parent)
        x = rng.random((B, N, V)) ** 4 + 1e-6
        p = x / x.sum(-1, keepdims=True)
        y = rng.random((B, N, V)) ** 4 + 1e-6
        qq = y / y.sum(-1, keepdims=True)
        tokens = rng.integers(0, V, (B, N))
        ua, ub = rng.random((B, N)), rng.random((B, N))
        v0, v1 = vocab_shard_range(V, rank, world)
        shard = _CpuShard(p[:, :, v0:v1], qq[:, :, v0:v1], v0, V, rank, world, tokens, parent, ua, ub)
        out = drive_vocab_shards([shard], _all_reduce_group(None), max_children(parent))[0]
        full = orc.verify_tree(p, qq, tokens, parent, None, ua, ub)
        for key in ("accept_len", "out_tokens", "out_nodes", "best_root"):     # every rank holds the whole result
            ok &= bool(np.array_equal(out[key].numpy(), full[key]))
    flags = [None] * world
    dist.all_gather_object(flags, ok)
    if rank == 0:
        q.put(all(flags))
    dist.barrier()
    dist.destroy_process_group()


def test_vocab_sharded_verify_protocol_over_gloo(m):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_vocab_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    ok = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok


# ---------------------------------------------------------------------------------------------------------
# bench.py --gpus N started by hand: it must start N ranks itself
# ---------------------------------------------------------------------------------------------------------
def _load_bench():
    import importlib.util
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    spec = importlib.util.spec_from_file_location("bench_under_test", os.path.join(root, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_bench_builds_the_launcher_command_for_n_ranks():
    bench = _load_bench()
    seen = []
    rc = bench.launch_ranks(4, ["--gpus", "4", "--steps", "2"], runner=lambda cmd: seen.append(cmd) or 0)
    assert rc == 0 and len(seen) == 1
    cmd = seen[0]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nnodes=1" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert 0 < int(cmd[cmd.index("--master-port") + 1]) < 65536
    assert cmd[-4:] == ["--gpus", "4", "--steps", "2"] and cmd[-5].endswith("bench.py")


_FAKE_RANK = """
import os, sys
import torch, torch.distributed as dist
dist.init_process_group("gloo")
t = torch.tensor([float(os.environ["RANK"]) + 1.0])
dist.all_reduce(t)
open(os.path.join(sys.argv[1], "rank%s" % os.environ["RANK"]), "w").write("%d %d %g" % (dist.get_world_size(), int(os.environ["LOCAL_RANK"]), t.item()))
dist.destroy_process_group()
"""


def test_bench_launcher_starts_two_real_ranks(tmp_path):
    """The launcher's command, run for real with a stand-in for the rank program: two processes that find each other
    over 127.0.0.1, see WORLD_SIZE = 2 and distinct LOCAL_RANKs."""
    bench = _load_bench()
    script = tmp_path / "fake_rank.py"
    script.write_text(_FAKE_RANK)
    rc = bench.launch_ranks(2, [str(tmp_path)], script=str(script))
    assert rc == 0
    got = sorted((tmp_path / ("rank%d" % r)).read_text() for r in range(2))
    assert got == ["2 0 3", "2 1 3"]


def test_bench_counts_the_rows_the_verify_kernel_reads():
    """verify_rows_read: an internal node's two rows once per rejected child, nothing for an accepted first child."""
    import torch
    bench = _load_bench()
    parent = parent_array(1, (3, 1))                  # root with three children, each with one child: 7 nodes
    N = len(parent)
    nxt = torch.full((2, N), -1, dtype=torch.int32)
    nxt[0, 0] = 1                                     # sequence 0: first child of the root accepted, its child rejected
    nxt[1, 0] = 3                                     # sequence 1: two rejections at the root, third child accepted ...
    nxt[1, 3] = 6                                     # ... and that child's only child accepted
    states = {"next_child": nxt, "c": torch.zeros((2, N), dtype=torch.float64)}
    rows, _ = bench.verify_rows_read(states, parent, np.array([N, N]))
    # sequence 0: root 0 rejections; nodes 1, 2, 3 each reject their one child -> 3 rejections
    # sequence 1: root 2 rejections; nodes 1, 2 reject their child (2), node 3 accepts (0)
    assert rows == 2 * (3 + 2 + 2)
    rows_cut, _ = bench.verify_rows_read(states, parent, np.array([4, 4]))     # level 2 sliced off: only the root counts
    assert rows_cut == 2 * (0 + 2)


def _enumerate_tiles(lens, n_act, units, stack, qb):
    """Brute force: (sequence, unit, query block, tile in item, queries, tiles in item) of every tile, in the
    kernel's order (prefix tiles before tree tiles inside an item)."""
    rows = []
    for b in range(len(lens)):
        L, Nb = int(lens[b]), int(n_act[b])
        if Nb <= 0:
            continue
        tkv = -(-L // 128) + -(-Nb // 128)
        nq = Nb * stack
        for h in range(units):
            for qi, q0 in enumerate(range(0, nq, qb)):
                for lt in range(tkv):
                    rows.append((b, h, qi, lt, min(qb, nq - q0), tkv))
    return np.array(rows, dtype=np.int64).reshape(-1, 6)


@pytest.mark.parametrize("seed", range(40))
def test_attention_plan_partitions_the_tiles_of_a_launch(m, seed):
    """mcsd_tree_attention_plan (the kernel's own work-partition functions, evaluated on the host): the blocks' ranges
    tile the launch without gaps, every probed tile is where a brute-force enumeration puts it, the block that the
    merging code computes for a tile is the block whose range holds it, no block's cost exceeds an even share by
    more than one heaviest tile, and in whole-item mode every block gets exactly one work item."""
    rng = np.random.default_rng(100 + seed)
    B = int(rng.choice([1, 2, 5, 16, 33, 256]))
    N = int(rng.choice([1, 15, 45, 82, 109, 128, 129, 160, 192]))
    H_kv = int(rng.choice([1, 2, 8]))
    G = int(rng.choice([1, 1, 2, 4, 8]))
    H_q = H_kv * G
    L_max = int(rng.choice([0, 100, 1000, 5000]))
    lens = rng.integers(0, L_max + 1, B).astype(np.int32)
    n_act = rng.integers(0, N + 1, B).astype(np.int32)
    if seed % 3 == 0:
        n_act[:] = N
    if seed == 5:                                   # a small launch: whole items
        B, lens, n_act = 1, np.array([min(L_max, 500)], dtype=np.int32), np.array([N], dtype=np.int32)
    n_blocks = int(rng.choice([1, 7, 148, 160]))
    assert m.mcsd_tree_attention_path(B, H_q, H_kv, N, 128, L_max, m.MCSD_BF16) == 1
    stack = next((s for s in (8, 4, 2) if G % s == 0 and s * N <= 160), 1)
    units = H_q // stack

    used, first, info, _ = m.mcsd_tree_attention_plan(B, H_q, H_kv, N, 128, L_max, m.MCSD_BF16, lens, n_act, n_blocks)
    total, total_cost, whole, qb = (int(x) for x in info)
    assert qb == (160 if N * stack > 128 else 128)          # trees wider than that are cut into query blocks of 160
    tiles = _enumerate_tiles(lens, n_act, units, stack, qb)
    assert total == len(tiles)
    assert first[0] == 0 and (np.diff(first) >= 0).all() and first[-1] == total
    assert (first[used:] == total).all()
    if total == 0:
        assert used == 0
        return
    assert 1 <= used <= n_blocks and (np.diff(first[: used + 1]) > 0).all()      # every used block owns a tile

    probes = np.unique(np.concatenate([first[:used], first[1: used + 1] - 1, rng.integers(0, total, 200)]))
    _, _, _, out = m.mcsd_tree_attention_plan(B, H_q, H_kv, N, 128, L_max, m.MCSD_BF16, lens, n_act, n_blocks, probes)
    assert (out[:, :6] == tiles[probes]).all()
    owner = np.searchsorted(first[1: used + 1], probes, side="right")            # block whose range holds the tile
    if whole:
        assert (out[:, 6] == -1).all()
        item_starts = np.flatnonzero(tiles[:, 3] == 0)
        assert used == len(item_starts) and (first[:used] == item_starts).all()
    else:
        assert (out[:, 6] == owner).all()
        # cost: block c's tiles cost (cost before its successor's first tile) - (cost before its own first tile)
        _, _, _, edge = m.mcsd_tree_attention_plan(B, H_q, H_kv, N, 128, L_max, m.MCSD_BF16, lens, n_act, n_blocks, first[:used])
        before = np.append(edge[:, 7], total_cost)
        assert (np.diff(before) > 0).all()
        heaviest = 64 + 256                                                       # a tile with an item's fixed cost on it
        assert np.diff(before).max() <= -(-total_cost // used) + heaviest
    # a tile number outside the launch is reported as such
    _, _, _, bad = m.mcsd_tree_attention_plan(B, H_q, H_kv, N, 128, L_max, m.MCSD_BF16, lens, n_act, n_blocks, [total, -1])
    assert (bad == -1).all()


def test_attention_plan_rejects_what_the_tensor_core_kernel_does_not_take(m):
    lens = np.array([10, 20], dtype=np.int32)
    with pytest.raises(m.McsdError):
        m.mcsd_tree_attention_plan(2, 4, 4, 15, 64, 128, m.MCSD_BF16, lens)                  # head_dim 64: CUDA-core kernel
    with pytest.raises(m.McsdError):
        m.mcsd_tree_attention_plan(2, 4, 4, 193, 128, 128, m.MCSD_BF16, lens)                # too many nodes
    with pytest.raises(ValueError):
        m.mcsd_tree_attention_plan(2, 4, 4, 15, 128, 128, m.MCSD_BF16, lens, n_blocks=161)
    assert int(m.lib.mcsd_tree_attention_plan(2, 4, 4, 15, 128, 128, m.MCSD_BF16, None, None, 4, None, None, 0, None, None)) == -1
