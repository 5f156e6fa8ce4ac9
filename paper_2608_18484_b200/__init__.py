"""SparsePR on B200: C-ABI CUDA library plus a thin Python binding.

Importing the package does not load the CUDA library; the first call into
`paper_2608_18484_b200.binding` does, and fails loudly if it is missing.
"""
__all__ = ["binding", "workloads"]
