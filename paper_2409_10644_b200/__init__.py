"""B200-native verification of a candidate token tree for multi-candidate speculative decoding.

The work is done by libmcsd.so (hand-written sm_100a kernels behind a C ABI, see include/mcsd.h);
this package is the thin binding with the same names.  The library is loaded on first use and a
missing build raises -- there is no fallback path.
"""
_BINDING_NAMES = (
    "McsdError", "TreeMask", "lib", "MCSD_BF16", "MCSD_F32", "MCSD_MAX_NODES",
    "mcsd_build_mask", "mcsd_tree_attention", "mcsd_tree_attention_workspace_bytes",
    "mcsd_verify_tree", "mcsd_verify_tree_logits", "mcsd_sample_roots", "mcsd_verify_tree_static", "mcsd_commit_kv", "layer_pointer_table", "mcsd_verify_tree_workspace_bytes", "mcsd_workspace_status", "verify_node_states", "mcsd_tree_attention_path", "mcsd_tree_attention_plan", "mcsd_selftest_bounded_wait",
    "mcsd_status_string", "mcsd_launch_count", "n_active_from_gamma", "shard_batch", "new_workspace",
    "VocabShard", "mcsd_verify_shard_workspace_bytes",
)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)


__all__ = list(_BINDING_NAMES)
