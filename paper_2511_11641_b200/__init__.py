"""libecospa: B200-native coupled-sparsity hot path (score, aligned top-k, compaction, compacted-pair GEMMs).

The work is done by CUDA kernels in libecospa.so behind a C ABI (include/ecospa.h);
`binding` marshals torch tensors into it.  Importing this package does not load the
library; the first call does, and raises if it has not been built.
"""
from . import algorithm1, binding, block, layers, workloads  # noqa: F401
