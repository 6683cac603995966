"""B200 (sm_100a) implementation of the NOVAK per-parameter optimizer step.

``binding`` wraps the C-ABI library (include/novak.h); ``optim`` is the
``torch.optim.Optimizer`` front end over it; ``workloads`` holds the
seeded synthetic parameter sets (shapes and value recipes only, none of the
method's arithmetic); ``build`` compiles the library in-tree with nvcc.
"""
from . import build  # noqa: F401

__all__ = ["build", "binding", "optim", "workloads"]
