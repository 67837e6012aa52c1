"""B200-native AdaComp hot path: worker-side SELECT_GRAD and the parameter-server
update of Algorithm 2, as a C-ABI CUDA library (``libadacomp``) with a thin ctypes
binding.

Nothing is imported eagerly: ``paper_1702_04683_b200.binding`` loads the CUDA
library (and fails loudly if it has not been built), ``workloads`` only generates
seeded synthetic inputs.
"""
__all__ = ["binding", "workloads", "build"]
__version__ = "0.1.0"
