"""Glenside access-pattern evaluation on B200 (sm_100a).

`synth` (seeded inputs, workload table) imports without the CUDA library;
`binding` loads the C-ABI shared library and raises if it is missing.
"""
__all__ = ["synth", "binding"]
