"""B200-native approximate query cache (PROXIMITY-FLAT) with an exact top-k corpus scan.

``paper_2503_05530_b200.prox`` is the binding of the CUDA library (it fails
loudly when the library is not built); ``paper_2503_05530_b200.workloads``
draws the seeded synthetic inputs.  Importing the package loads neither.
"""
__all__ = ["prox", "workloads"]
