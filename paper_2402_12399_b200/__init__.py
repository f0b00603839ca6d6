"""Rectify-Router MoE layer (arXiv 2402.12399) for B200: a C-ABI CUDA library
(librr.so, declared in include/rr.h) and this thin binding.

`synth` (seeded input generators) imports without the CUDA library; everything in
`binding` needs librr.so and raises if it is missing.
"""
from . import synth  # noqa: F401

_BINDING = ("IR", "FR", "SCORE", "FR_SOFTMAX", "LOCAL_CAP", "GRAD_EXACT", "BF16", "F32", "RRError", "RouteTables", "alloc_tables",
            "alloc_workspace", "route_workspace_bytes", "route", "route_noalloc", "check", "moe_workspace_bytes",
            "moe_fwd", "moe_bwd", "gate_workspace_bytes", "gate_fwd", "gate_bwd", "aux_workspace_bytes",
            "aux_loss_fwd", "aux_loss_bwd", "gate_route", "gate_route_workspace_bytes", "route_loss", "route_loss_workspace_bytes", "test_set_wait_limit_ns", "Trace", "status_string", "lib",
            "LIB_PATH")


def __getattr__(name):
    if name in _BINDING or name == "binding":
        import importlib
        binding = importlib.import_module(__name__ + ".binding")
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(name)
