"""B200-native DEFT gradient-selection hot path (C-ABI CUDA library + thin binding).

``paper_2307_03500_b200.deft`` is the binding over ``libdeft.so``;
``paper_2307_03500_b200.workloads`` draws the seeded synthetic inputs.  Nothing is
imported eagerly so that the input generators can be used without the library.
"""
__all__ = ["deft", "workloads", "build"]
