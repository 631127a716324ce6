"""B200-native population replay of the GORGO routing cost model.

``paper_2602_11688_b200.binding`` exposes the C-ABI entry points of ``libgorgo_b200.so``
(it raises if the library has not been built); ``paper_2602_11688_b200.workloads``
generates the seeded synthetic traces.
"""
__all__ = ["binding", "workloads", "build"]
