"""B200 (sm_100a) routed-LoRA library: Python binding over the C ABI declared in include/molora.h.

The binding only marshals arguments (device pointers, sizes, the current CUDA stream); every step of
the path -- routing, grouping, shrink/expand -- runs in the library's own kernels.  There is no CPU or
PyTorch fallback: if the shared library is missing or a call is refused, an exception is raised.
"""
from .binding import (  # noqa: F401
    MoloraError, lib_path, load_library, exported_symbols,
    molora_version, molora_status_string, molora_launch_count, molora_debug_set, TUNING_NAMES,
    molora_route_vocab, molora_route_composite, molora_route_mlp, molora_route_mlp_workspace_bytes, molora_route_gate, molora_route_gate_workspace_bytes, molora_route_gate_noalloc, molora_route_gate_prepare, molora_route_mlp_prepare, molora_selftest_bounded_wait,
    molora_group_workspace_bytes, molora_group,
    molora_apply_workspace_bytes, molora_apply, molora_apply_batched, molora_group_apply_batched, molora_topk_softmax, molora_apply_topk,
    ProjDesc, F32, BF16, HotSet, molora_route_hotset,
    HostProj, molora_forward_host, molora_forward_host_arena_bytes, ROUTE_VOCAB, ROUTE_GATE, ROUTE_GIVEN,
)
