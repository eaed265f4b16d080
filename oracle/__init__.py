"""TEST INFRASTRUCTURE: the CPU oracle.

A plain, slow, fp64/int CPU implementation of what the tagged recursive
dataflow path computes, written from the paper: the Section 3 graph
transformation (`transform`), a literal tagged-token interpreter (`tagged`),
and direct recursive evaluation with reverse-recursion gradients (`direct`).
It shares no code with the CUDA path and must not be imported by it; only
tests, the smoke check and the CPU-baseline leg of the benchmark use it.
"""
