"""Batched simulator of straggling distributed-SGD variants (K-sync, K-batch-sync, K-async,
K-batch-async, growing-K schedule) on one B200: CUDA kernels behind a C-ABI library, plus a thin
ctypes binding.  ``inputs`` only makes seeded synthetic data; ``binding`` loads the library and
fails loudly if it has not been built (there is no CPU path)."""

__all__ = ["inputs", "binding", "build"]
