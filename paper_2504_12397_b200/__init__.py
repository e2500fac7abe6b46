"""B200-native aLoRA suffix-prefill hot path: CUDA kernels behind a C ABI plus a thin binding.

`paper_2504_12397_b200.binding` loads the compiled library and fails loudly when it is missing;
`paper_2504_12397_b200.workloads` draws seeded synthetic inputs and touches neither.
"""
__all__ = ["binding", "workloads", "build"]
