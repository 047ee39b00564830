"""The workspace-free verify entry point (for callers that cannot allocate device memory when they call)
must give exactly the results of the regular entry point, call after call, although every call reuses the
same built-in scratch array.  Collected last on purpose."""
import dataclasses

import numpy as np
import pytest
import torch

from mcsd_inputs import gammas, parent_array, verify_inputs, workload
from oracle import mcsd_oracle as orc
from tests.helpers import condition_uniforms, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def m():
    from paper_2409_10644_b200 import build
    build.build()
    import paper_2409_10644_b200 as pkg
    return pkg


def _outputs(B, n_levels, R, dev):
    return {
        "accept_len": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "out_tokens": torch.full((B, n_levels + 1), -7, dtype=torch.int32, device=dev),
        "out_nodes": torch.full((B, n_levels), -7, dtype=torch.int32, device=dev),
        "best_root": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "next_roots": torch.full((B, R), -7, dtype=torch.int32, device=dev),
    }


def test_static_scratch_entry_point_matches_the_workspace_one_twice_in_a_row(m):
    dev = torch.device("cuda", 0)
    R = 4
    # two different problems back to back: a large one, then a smaller one that leaves most of the
    # previous call's node states behind in the shared array
    cases = [(workload(5), 12, 4000, 0), (workload(3), 5, 1000, 1)]
    for w, B, V, step in cases:
        parent = parent_array(w.n_roots, w.branching)
        tm = m.mcsd_build_mask(parent, device=dev)
        vin = verify_inputs(w, step, dev, parent=parent, B=B, V=V)
        gam_h = gammas(dataclasses.replace(w, B=B), step)
        gam = torch.from_numpy(gam_h).to(dev)
        # uniforms kept clear of the oracle's thresholds, so that the oracle's integers are the expected ones too
        host = {k: to_np(v) for k, v in vin.items()}
        ua, ub = condition_uniforms(host["p"], host["q"], host["tokens"], parent, gam_h, host["u_accept"], host["u_bonus"])
        ua_d, ub_d = torch.from_numpy(ua).to(dev), torch.from_numpy(ub).to(dev)
        ref = m.mcsd_verify_tree(vin["p"], vin["q"], vin["tokens"], tm, gam, ua_d, ub_d, R=R)
        out = _outputs(B, tm.n_levels, R, dev)
        got = m.mcsd_verify_tree_static(vin["p"], vin["q"], vin["tokens"], tm, gam, ua_d, ub_d, out, R=R)
        torch.cuda.synchronize()
        for k in ("accept_len", "out_tokens", "out_nodes", "best_root", "next_roots"):
            assert torch.equal(got[k], ref[k]), k          # integer results: identical, not just close
        # and directly against the CPU oracle, not only against the other entry point
        exp = orc.verify_tree(host["p"], host["q"], host["tokens"], parent, gam_h, ua, ub, R=R)
        for k in ("accept_len", "out_tokens", "out_nodes", "best_root", "next_roots"):
            assert np.array_equal(got[k].cpu().numpy(), exp[k]), k
        assert int(ref["accept_len"].max()) >= 0


def test_static_scratch_entry_point_rejects_oversized_problems(m):
    import ctypes
    fake = ctypes.c_void_p(0x1000)     # never dereferenced: the size check comes first
    st = m.lib.mcsd_verify_tree_static(fake, fake, fake, fake, fake, 4, 1, None, fake, fake, 200, 192, 100,
                                       fake, fake, fake, fake, None, 0, None)
    assert st == -8
    assert "built-in scratch" in m.mcsd_status_string(st)
