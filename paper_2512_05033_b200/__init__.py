"""B200-native hot path of step-level speculative generation with an advantage-aware router:
paged grouped-query attention (decode and step chunks), the router head and step rollback.

``paper_2512_05033_b200.binding`` is the ctypes binding of the C-ABI library (``csrc/``);
``paper_2512_05033_b200.workloads`` draws the seeded synthetic inputs.  Importing the package loads
neither; importing ``binding`` fails loudly if the CUDA library has not been built.
"""
__all__ = ["binding", "workloads", "build"]
