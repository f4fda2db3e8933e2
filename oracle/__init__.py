"""CPU oracle for tensorized attention (fp64).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
The CUDA library never imports, links or calls anything here, and nothing here imports the
CUDA package.
"""
from .ta_oracle import (  # noqa: F401
    backward,
    dense_effective_matrix,
    dense_hop_matrix,
    forward,
    forward_dense,
    num_threads,
)
