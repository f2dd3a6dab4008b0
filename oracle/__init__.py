"""fp64 CPU oracle of the USV sparsified-attention path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
cpu-baseline / reference legs.  The CUDA library and its Python binding never import it.
"""
from .usv_oracle import *  # noqa: F401,F403
