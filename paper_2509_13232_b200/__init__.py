"""B200-native SPO (Single-stream Policy Optimization) hot path.

`binding` wraps the C-ABI library (libspo.so) one to one; `inputs` draws the
seeded synthetic workloads.  Nothing here computes on the CPU: every step of
the path runs in the CUDA kernels behind the C ABI, and calling into the
binding without a built library raises.
"""

__all__ = ["binding", "inputs", "build"]
