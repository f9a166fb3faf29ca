"""CPU checker (test infrastructure only): numpy/ctypes front end of capmoe_oracle.cpp.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark import
this package.  It never imports the CUDA binding.
"""
from .oracle import *  # noqa: F401,F403
