"""B200-native batched draft-verification pass of confidence-gated cascaded verification.

The package is a thin Python layer over libconfspec.so (hand-written sm_100a CUDA behind a C ABI, declared in
include/confspec.h). Nothing here computes: `binding` marshals arguments, `runner` wires a seeded workload to
the C calls.
"""
from . import binding
from .binding import ConfSpecError, load_library
from .runner import VerifySession

__all__ = ["binding", "ConfSpecError", "load_library", "VerifySession"]
