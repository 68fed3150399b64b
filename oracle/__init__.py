"""ORACLE: a plain, slow CPU implementation of the straggler-SGD simulation, written from the
paper's definitions.  It is test infrastructure: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the CUDA library and its Python binding never do, and
the two share no code.

  core    Philox4x32-10, deterministic -ln(u), delays, minibatch indices, bulk arrival process (C)
  models  per-minibatch loss and gradient of the four models (numpy, fp64)
  sim     event-driven simulator of one replica (Python, interleaves arrivals and updates)
  curves  error against wall clock on a common time grid
"""
from . import core, curves, models, sim  # noqa: F401
from .sim import OracleReplica  # noqa: F401
