"""B200-native fused credit-assignment scans (GAE, V-Trace, Retrace(lambda), TD(lambda),
discounted returns, eligibility traces, episodic prefix sums) behind a small C ABI.

``workloads`` holds the seeded synthetic input generators; ``binding`` is the thin ctypes layer
over ``librlcs.so`` (argument marshalling only -- every step runs in the CUDA kernels; there is no
CPU fallback, and calling into the binding without the built library raises).
``api`` offers the same calls under the paper's ``compute_*`` names, choosing the entry point from dtype
and layout.
"""
__all__ = ["api", "binding", "workloads", "build"]
