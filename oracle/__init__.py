"""CPU oracle for the Longest-Stable-Prefix decode path.

TEST INFRASTRUCTURE ONLY.  A plain, slow numpy/fp64 restatement of what the path computes,
written from the paper's algorithm and formulas.  It shares no code with the CUDA library,
never imports it, and must not be imported by the product path: only the tests, the smoke
check and the benchmark's CPU-baseline leg may use it.

Parity status of each part (what pins it besides itself) is listed in each module header.
"""
