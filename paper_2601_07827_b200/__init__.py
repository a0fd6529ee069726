"""B200-native general binary tensor contraction, D = alpha * op(A) * op(B) + beta * op(C).

`paper_2601_07827_b200.api` is the Python binding of the C-ABI library (it loads the CUDA
shared library and fails loudly when that is missing); `paper_2601_07827_b200.inputs` creates
the seeded synthetic workloads.  Nothing is imported eagerly so that the input generators can
be used without touching the GPU library.
"""
__all__ = ["api", "inputs"]
