"""B200-native (sm_100a) FlashLoop loop-r prefill step: a C-ABI CUDA library and its thin binding.

`from paper_2609_29812_b200 import binding` loads the shared library (and fails loudly if it has
not been built); `workloads` holds the seeded synthetic input generators.
"""
__all__ = ["binding", "workloads", "build"]
