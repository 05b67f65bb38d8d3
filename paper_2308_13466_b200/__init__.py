"""B200-native (sm_100a) hot path of SAT, staleness-alleviated training for partition-parallel GNNs
(arXiv 2308.13466): halo pull from the historical-embedding cache, LSTM-GCN embedding predictor,
fused CSR SpMM + dense transform forward, backward, cache push — as a C-ABI CUDA library
(`libsat_b200.so`, declared in include/sat_b200.h) with a thin ctypes binding of the same names.

There is no CPU implementation in this package: importing `binding` fails loudly when the
library is missing.
"""
from .build import build, lib_path  # noqa: F401

__all__ = ["build", "lib_path"]
