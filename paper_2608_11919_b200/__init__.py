"""B200-native fused global-norm clip + block-wise 8-bit AdamW optimizer step.

The product is the C-ABI CUDA library `liblt_hybrid8.so` (declared in include/lt.h, built in-tree by
`python -m paper_2608_11919_b200.build`); this package is a thin ctypes binding with the same
entry-point names plus seeded synthetic workloads. There is no CPU or PyTorch fallback: the first use
of any entry point loads the library and raises ImportError if it has not been built.
(`paper_2608_11919_b200.build` and `.workloads` import without the library.)
"""
_BINDING_NAMES = (
    "LT_F32", "LT_BF16", "LtError", "HParams", "TensorList", "library_path",
    "lt_hybrid8_state_bytes", "lt_hybrid8_code_table", "lt_workspace_bytes", "lt_hybrid8_state_init",
    "lt_grad_sqnorm_multi", "lt_grad_sqnorm_multi_noalloc", "lt_grad_sqnorm_per_tensor", "lt_skip_count_update", "lt_hybrid8_step", "lt_status_str",
    "Hybrid8Optimizer", "GraphedHybrid8Optimizer", "lt_step_state_advance", "lt_hybrid8_step_graph",
)
__all__ = list(_BINDING_NAMES)


def __getattr__(name):
    if name in _BINDING_NAMES:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
