"""B200 (sm_100a) implementation of ToMA's per-block token-reduction path.

`paper_2509_10918_b200.binding` holds the ctypes binding of the C-ABI library
(declared in include/toma.h); its names are re-exported here lazily so that
`paper_2509_10918_b200.build` can be imported before the library exists.
"""
import importlib

_BINDING_NAMES = {
    "TomaDesc", "TomaError", "make_desc", "desc_from_config", "torch_dtype", "toma_validate", "toma_workspace_bytes",
    "toma_weights_bytes", "toma_dest_per_tile", "toma_launch_counter", "toma_status_str", "toma_select", "toma_select_static", "toma_merge_weights", "toma_merge",
    "toma_unmerge", "toma_attention", "toma_attention_workspace_bytes", "toma_attention_plan", "toma_test_set_tuning", "toma_test_wait_timeout", "toma_block", "toma_block_host", "toma_linear", "toma_block_proj", "toma_attention_proj", "toma_attention_proj_workspace_bytes", "toma_block_mlp", "toma_mlp", "toma_mlp_workspace_bytes", "toma_weights_export", "toma_weights_import", "toma_unmerge_weights_export", "UNMERGE_MODES", "alloc_workspace",
    "alloc_weights", "alloc_idx", "EXPORTS", "LIB_PATH", "lib", "TOMA_BF16", "TOMA_F32",
}


def __getattr__(name):
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(".binding", __name__), name)
    raise AttributeError(name)
