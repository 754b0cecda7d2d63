"""CPU checker written from the paper (test infrastructure only).

`interp` is a numpy interpreter of access-pattern programs; `brute` wraps
brute.c, the paper's element-wise equations as nested C loops.  Only tests,
the smoke check and the benchmark's CPU-baseline leg may import this package.
"""
