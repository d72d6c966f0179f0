"""B200-native AudioKV eviction pass: CUDA kernels behind a C-ABI library plus a thin Python binding.

`paper_2604_06694_b200.binding` loads the CUDA library (and fails loudly when it is missing);
`paper_2604_06694_b200.workloads` draws the seeded synthetic inputs and imports no CUDA code.
"""
__all__ = ["binding", "workloads"]
