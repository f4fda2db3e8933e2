"""Tensorized attention (arxiv 2410.20926, Algorithm 1) for NVIDIA B200: Python binding of the
C-ABI CUDA library.  See ``api`` for the calls and ``inputs`` for the seeded synthetic data."""
