"""B200-native precision-switch search of AdaPT (per-layer <WL,FL> search).

The compute lives in ``csrc/`` (CUDA kernels behind a C-ABI shared library);
``binding`` marshals arguments to it and ``workloads`` makes seeded inputs.
"""
from . import workloads  # noqa: F401
