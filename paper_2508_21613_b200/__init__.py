"""B200-native real-time execution-plan search (Chameleon, Section "Planner" / "Estimator").

The product is the C-ABI library ``libchameleon.so`` (hand-written sm_100a CUDA);
``binding`` is a thin ctypes shim over it and ``workloads`` draws seeded synthetic
inputs.  Nothing here computes on the CPU: if the CUDA library is missing, the
binding raises.
"""

__all__ = ["binding", "workloads", "build"]
