"""B200-native Dynamic Vocabulary Pruning hot path (arXiv 2512.23087).

The work is done by hand-written CUDA kernels for sm_100a behind a C-ABI
library (``include/dvp.h``); ``binding`` marshals arguments to it and
``inputs`` builds seeded synthetic workloads.  Importing this package does not
load the library; the first call into ``binding`` does, and fails loudly if the
library has not been built.
"""
__all__ = ["binding", "inputs", "build"]
