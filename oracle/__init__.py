"""CPU oracle of the ViTCoP pruning operator chain -- TEST INFRASTRUCTURE ONLY.

``vitcop_oracle.cpp`` is the plain fp64 statement of the paper's equations and
algorithms; this package compiles it on first use (g++, host-specific flags, so
the shared object is rebuilt on every new machine) and exposes thin numpy
wrappers.  Nothing here imports or is imported by the CUDA package.
"""
from .api import *  # noqa: F401,F403
