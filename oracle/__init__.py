"""CPU oracle of the sparsity-aware IVFPQ query path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do.
"""

from .cpu_oracle import build, coarse, entry_stats, num_threads, search, set_num_threads, thresholds, thresholds_knn

__all__ = ["build", "coarse", "entry_stats", "num_threads", "search", "set_num_threads", "thresholds", "thresholds_knn"]
