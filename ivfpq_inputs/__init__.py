"""Seeded synthetic inputs for the sparsity-aware IVFPQ query path.

This package is test/bench infrastructure shared by the CPU oracle's tests and
by the CUDA library's tests: it draws the synthetic base vectors and queries,
trains and encodes an IVFPQ index from them (the paper's offline phase,
Algorithm 1, without the ray-tracing scene and without the entry->points map),
calibrates hit radii, builds the density maps and the polynomial regressor of the dynamic
threshold, computes exact brute-force neighbours for recall, and
reads/writes the index file.  It contains none of the online search steps
(coarse probe selection, selective look-up table, list scan, top-k): those live
in `oracle/` (CPU) and in the CUDA library, which share no code.
"""

from .configs import CONFIGS, WorkloadConfig, get_config
from .generators import MixtureSpec, make_mixture, sample_mixture
from .index_build import (
    IvfPqIndex,
    build_index,
    build_index_streamed,
    calibrate_radius,
    calibrate_radius_ip,
    lossless_toy_index,
    load_index,
    save_index,
)
from .groundtruth import exact_knn, recall_at_k, recall_1_at_k
from .thresholds import (DensityAccumulator, ThresholdModel, containing_thresholds, density_maps,
                         fit_threshold_model)

__all__ = [
    "CONFIGS",
    "WorkloadConfig",
    "get_config",
    "MixtureSpec",
    "make_mixture",
    "sample_mixture",
    "IvfPqIndex",
    "build_index",
    "build_index_streamed",
    "calibrate_radius",
    "calibrate_radius_ip",
    "lossless_toy_index",
    "load_index",
    "save_index",
    "exact_knn",
    "recall_at_k",
    "recall_1_at_k",
    "ThresholdModel",
    "containing_thresholds",
    "DensityAccumulator",
    "density_maps",
    "fit_threshold_model",
]
