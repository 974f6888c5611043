"""B200-native plasticity evaluation (SP loss + freezing rule) -- Python binding.

The compute lives in the CUDA library behind the C ABI declared in
``include/egeria.h``; :mod:`paper_2201_06227_b200.binding` only marshals
arguments.  :mod:`paper_2201_06227_b200.workloads` draws seeded synthetic inputs.
"""
__all__ = ["binding", "workloads"]
