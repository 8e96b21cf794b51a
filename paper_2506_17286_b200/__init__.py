"""B200-native GTA (Grouped-head latenT Attention) operator: causal prefill, single-token
decode and cache append, as hand-written sm_100a CUDA kernels behind a C-ABI library.

`paper_2506_17286_b200.inputs` (synthetic input recipes) imports without the CUDA library;
the operator entry points live in `paper_2506_17286_b200.binding` and raise if the library
has not been built.
"""
__all__ = ["inputs", "binding"]
