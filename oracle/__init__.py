"""CPU oracle for mixed-precision KV-cache quantization (test infrastructure).

A plain, slow NumPy restatement of what the path computes: group-wise
asymmetric round-to-nearest quantization of K and V at independent bit widths
(the uniform scalar quantizer of App. B.1 applied per group with a minimum
offset), the packed page format, the dequantizer, and softmax attention
(App. A.1 notation: S = QK^T/sqrt(d), A = softmax(S), output A V) in fp64 over
the dequantized cache.

This package is test infrastructure only.  It shares no code with the CUDA
library and must never be imported by the product path; only tests, the smoke
check and the benchmark's CPU-baseline leg use it.

Parity status: every function here is pinned by the CPU test-suite to closed
forms, invariants, brute force or a library routine.  Parity unpinned: the
paper's absolute MSE / accuracy table values (they need its models and
datasets); nothing in this package claims to reproduce them.
"""
from . import quantizer, layout, attention, cache, error  # noqa: F401
