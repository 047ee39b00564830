"""Test-side glue: runs the CPU oracle on generated inputs and conditions uniforms on its thresholds."""
import numpy as np
import torch

from mcsd_inputs import UNIFORM_MARGIN
from oracle import mcsd_oracle as orc


def to_np(t):
    return t.detach().float().cpu().numpy() if t.dtype in (torch.bfloat16, torch.float32) else t.detach().cpu().numpy()


def condition_uniforms(p, q, tokens, parent, gamma, u_accept, u_bonus, seed=12345, margin=UNIFORM_MARGIN, max_rounds=50):
    """Redraw (seeded) every uniform that lies within `margin` of a decision threshold the oracle evaluates.

    Inputs and outputs are numpy arrays (p, q fp32; uniforms fp32).  The thresholds come from the oracle
    only; nothing here looks at a GPU result."""
    rng = np.random.default_rng(seed)
    ua = np.array(u_accept, dtype=np.float32, copy=True)
    ub = np.array(u_bonus, dtype=np.float32, copy=True)
    for _ in range(max_rounds):
        m_acc, m_bon = orc.decision_margins(p, q, tokens, parent, gamma, ua, ub)
        bad_a = m_acc < margin
        bad_b = m_bon < margin
        if not bad_a.any() and not bad_b.any():
            return ua, ub
        ua[bad_a] = rng.uniform(margin, 1 - margin, size=int(bad_a.sum())).astype(np.float32)
        ub[bad_b] = rng.uniform(margin, 1 - margin, size=int(bad_b.sum())).astype(np.float32)
    raise RuntimeError("could not move the uniforms away from the thresholds")


def oracle_attention_rows(inp, seq_lens, n_active, parent, scale, pairs):
    """Oracle tree attention for the listed (b, h) pairs only; returns {(b, h): [N][D] fp64}."""
    out = {}
    for (b, h) in pairs:
        sl = lambda k: to_np(inp[k][b:b + 1, h:h + 1])
        na = None if n_active is None else [int(n_active[b])]
        o = orc.tree_attention(sl("q"), sl("k_cache"), sl("v_cache"), sl("k_tree"), sl("v_tree"),
                               [int(seq_lens[b])], na, parent, scale)
        out[(b, h)] = o[0, 0]
    return out
