"""B200-native halted-prefill hot path of DASH (Delta Attention Selective Halting).

``paper_2604_18103_b200.dash`` is the thin binding over the C-ABI CUDA library
(loaded on first use; it raises if the library is missing -- there is no CPU
fallback).  ``paper_2604_18103_b200.workloads`` only draws seeded inputs.
"""
