"""The C ABI library loads, exports every declared symbol, and rejects bad arguments on the host
before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def m():
    from paper_2409_10644_b200 import build
    build.build()
    import paper_2409_10644_b200 as pkg
    return pkg


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mcsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mcsd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(m):
    names = _declared_functions()
    assert {"mcsd_build_mask", "mcsd_tree_attention", "mcsd_verify_tree"} <= set(names)
    for n in names:
        assert hasattr(m.lib, n), n


def test_status_strings(m):
    seen = {m.mcsd_status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert m.mcsd_status_string(-99) == "unknown status"


FAKE = ctypes.c_void_p(0x1000)      # never dereferenced: every call below fails its checks first


def test_build_mask_rejects_bad_trees_on_the_host(m):
    def call(parent, n=None, words=1):
        arr = np.asarray(parent, dtype=np.int32)
        return m.lib.mcsd_build_mask(arr.ctypes.data_as(ctypes.c_void_p), len(arr) if n is None else n, FAKE, words,
                                     FAKE, FAKE, None, None, None)
    assert call([-1, 1]) == -3              # parent not earlier
    assert call([-1, 0, 1, 0]) == -3        # depth decreases / children not contiguous
    assert call([-1, -1, 1, 0]) == -3
    assert call([0, -1]) == -3              # node 0 must be a root
    assert call([-1, -2]) == -3
    assert call([-1], n=0) == -2
    assert call([-1] * 193) == -2
    assert call([-1] * 65, words=1) == -2   # 65 nodes need two words
    assert m.lib.mcsd_build_mask(None, 1, FAKE, 1, FAKE, FAKE, None, None, None) == -1


def test_attention_argument_checks(m):
    L = m.lib
    ws = L.mcsd_tree_attention_workspace_bytes
    assert ws(1, 4, 15, 64, 128, m.MCSD_F32) >= 256
    assert ws(1, 4, 15, 96, 128, m.MCSD_F32) == 0          # head_dim must be 64 or 128
    assert ws(1, 4, 193, 64, 128, m.MCSD_F32) == 0
    assert ws(1, 4, 15, 64, 128, 7) == 0

    def call(q=FAKE, B=1, H=4, N=15, D=64, Lm=128, dtype=1, wsp=FAKE, wsb=1 << 30, words=1):
        return L.mcsd_tree_attention(q, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, words, B, H, N, D, Lm,
                                     ctypes.c_float(0.125), dtype, wsp, wsb, None)
    assert call(q=None) == -1
    assert call(D=96) == -2
    assert call(N=0) == -2
    assert call(N=193) == -2
    assert call(dtype=5) == -4
    assert call(wsb=16) == -5
    assert call(wsp=ctypes.c_void_p(0x1010)) == -2      # workspace must be 256-byte aligned
    assert call(N=100, words=1) == -2


def test_attention_gqa_argument_checks(m):
    L = m.lib

    def call(Hq=8, Hkv=2, q=FAKE, wsb=1 << 30):
        return L.mcsd_tree_attention_gqa(q, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, FAKE, 1, 1, Hq, Hkv, 15, 64, 128,
                                         ctypes.c_float(0.125), 1, FAKE, wsb, None)
    assert call(Hq=8, Hkv=3) == -2              # query heads must be a multiple of the key/value heads
    assert call(Hkv=0) == -2
    assert call(Hq=2, Hkv=4) == -2
    assert call(q=None) == -1
    assert call(wsb=16) == -5


def test_verify_argument_checks(m):
    L = m.lib
    assert L.mcsd_verify_tree_workspace_bytes(16, 45, 32000) >= 256 + 16 * 45 * 16

    def call(p=FAKE, B=2, N=15, V=100, nl=4, nr=1, R=0, wsb=1 << 20, nxt=None):
        return L.mcsd_verify_tree(p, FAKE, FAKE, FAKE, FAKE, nl, nr, None, FAKE, FAKE, B, N, V, FAKE, FAKE, FAKE, FAKE,
                                  nxt, R, FAKE, wsb, None)
    assert call(p=None) == -1
    assert call(N=193) == -2
    assert call(V=0) == -2
    assert call(nl=0) == -2
    assert call(nr=0) == -2
    assert call(R=33, nxt=FAKE) == -2
    assert call(R=2, nxt=None) == -1
    assert call(wsb=8) == -5


def test_verify_shard_argument_checks(m):
    L = m.lib
    assert L.mcsd_verify_shard_workspace_bytes(16, 45) >= 256 + 16 * 45 * (16 + 24) + 16 * 8
    assert L.mcsd_verify_shard_workspace_bytes(0, 45) == 0

    def gather(p=FAKE, B=2, N=15, Vs=50, v0=0, Vt=100, nl=4):
        return L.mcsd_verify_shard_gather(p, FAKE, FAKE, FAKE, FAKE, nl, None, B, N, Vs, v0, Vt, FAKE, None)
    assert gather(p=None) == -1
    assert gather(N=193) == -2
    assert gather(Vs=0) == -2
    assert gather(v0=60) == -2               # columns 60..110 of a 100-id vocabulary
    assert gather(v0=-4) == -2
    assert gather(nl=0) == -2

    def rnd(y=FAKE, rd=0, B=2, N=15, Vs=50, wsb=1 << 20):
        return L.mcsd_verify_shard_round(FAKE, FAKE, FAKE, FAKE, 4, None, FAKE, FAKE, y, rd, B, N, Vs, FAKE, wsb, None)
    assert rnd(y=None) == -1
    assert rnd(rd=-1) == -2
    assert rnd(rd=16) == -2
    assert rnd(B=0) == -2
    assert rnd(wsb=64) == -5

    def select(mass=FAKE, rank=0, world=2, nr=1, wsb=1 << 20):
        return L.mcsd_verify_shard_select(FAKE, FAKE, FAKE, 4, nr, 2, 15, 50, 0, 100, rank, world, FAKE, FAKE, FAKE, FAKE,
                                          mass, FAKE, wsb, None)
    assert select(mass=None) == -1
    assert select(rank=2) == -2
    assert select(world=0) == -2
    assert select(nr=0) == -2
    assert select(wsb=64) == -5

    def pick(u=FAKE, rank=1, world=2, wsb=1 << 20):
        return L.mcsd_verify_shard_pick(FAKE, FAKE, u, 4, 2, 15, 50, 50, 100, rank, world, FAKE, FAKE, FAKE, wsb, None)
    assert pick(u=None) == -1
    assert pick(rank=-1) == -2
    assert pick(world=2000) == -2
    assert pick(wsb=64) == -5


def test_verify_logits_argument_checks(m):
    L = m.lib

    def call(zt=FAKE, zd=FAKE, dtype=1, T=0.7, ua=FAKE, B=2, N=15, V=100, nl=4, nr=1, R=0, wsb=1 << 20, nxt=None):
        return L.mcsd_verify_tree_logits(zt, zd, dtype, ctypes.c_float(T), FAKE, FAKE, FAKE, nl, nr, None, ua, FAKE,
                                         B, N, V, FAKE, FAKE, FAKE, FAKE, nxt, R, FAKE, wsb, None)
    assert call(zt=None) == -1
    assert call(zd=None) == -1                   # the draft logits are needed unless the temperature is 0
    assert call(ua=None) == -1
    assert call(T=-1.0) == -2
    assert call(T=float("nan")) == -2
    assert call(T=1e-5) == -2
    assert call(dtype=9) == -4
    assert call(N=193) == -2
    assert call(V=0) == -2
    assert call(R=2, nxt=None) == -1
    assert call(wsb=8) == -5
    assert call(T=0.0, zd=None, ua=None, wsb=8) == -5    # greedy passes the pointer checks without draft and uniforms


def test_sample_roots_argument_checks(m):
    L = m.lib

    def call(p=FAKE, B=2, N=15, V=100, nl=4, R=2, wsb=1 << 20, u=FAKE):
        return L.mcsd_sample_roots(p, FAKE, FAKE, FAKE, FAKE, nl, u, B, N, V, R, FAKE, FAKE, wsb, None)
    assert call(p=None) == -1
    assert call(u=None) == -1
    assert call(R=0) == -2
    assert call(R=33) == -2
    assert call(N=193) == -2
    assert call(nl=0) == -2
    assert call(wsb=8) == -5

    def call_l(T=0.7, dtype=1, zd=FAKE):
        return L.mcsd_sample_roots_logits(FAKE, zd, dtype, ctypes.c_float(T), FAKE, FAKE, FAKE, 4, FAKE, 2, 15, 100, 2,
                                          FAKE, FAKE, 8, None)
    assert call_l() == -5
    assert call_l(T=0.0) == -2                  # greedy verification has nothing to sample
    assert call_l(dtype=7) == -4
    assert call_l(zd=None) == -1


def test_commit_kv_argument_checks(m):
    L = m.lib

    def call(kc=FAKE, n_layers=2, B=2, H=2, N=15, D=64, Lm=64, dtype=1, nl=4):
        return L.mcsd_commit_kv(kc, FAKE, FAKE, FAKE, n_layers, FAKE, FAKE, FAKE, FAKE, nl, B, H, N, D, Lm, dtype, None)
    assert call(kc=None) == -1
    assert call(n_layers=0) == -2
    assert call(D=96) == -2
    assert call(N=193) == -2
    assert call(nl=0) == -2
    assert call(dtype=3) == -4


def test_attention_kernel_choice_is_a_documented_function_of_the_shape(m):
    """mcsd_tree_attention_path: the tensor-core kernel's limits (bf16, head_dim 128, at most 256 sequences, 32-bit
    per-sequence tile tables) are checked on the host; everything else valid runs the CUDA-core kernel."""
    bf16, f32 = m.MCSD_BF16, m.MCSD_F32
    path = m.mcsd_tree_attention_path
    assert path(16, 32, 32, 45, 128, 4096, bf16) == 1
    assert path(32, 32, 32, 160, 128, 4096, bf16) == 1
    assert path(1, 32, 8, 45, 128, 512, bf16) == 1                 # grouped queries
    assert path(1, 4, 4, 15, 64, 128, f32) == 0                    # fp32
    assert path(2, 4, 4, 45, 64, 512, bf16) == 0                   # head_dim 64
    assert path(256, 8, 8, 45, 128, 4096, bf16) == 1
    assert path(257, 8, 8, 45, 128, 4096, bf16) == 0               # more sequences than the per-sequence tables hold
    # the tile tables are 32-bit: B * (L_max / 128 + 4) must stay below 2^23
    assert path(256, 1, 1, 45, 128, 4_000_000, bf16) == 1
    assert path(256, 1, 1, 45, 128, 4_300_000, bf16) == 0
    assert path(2, 1, 1, 192, 128, 500_000_000, bf16) == 1
    assert path(2, 1, 1, 192, 128, 600_000_000, bf16) == 0
    with pytest.raises(m.McsdError):
        path(1, 4, 4, 193, 128, 128, bf16)                         # more nodes than a tree may have
    with pytest.raises(m.McsdError):
        path(1, 6, 4, 45, 128, 128, bf16)                          # query heads not a multiple of key/value heads
