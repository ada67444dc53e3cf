"""Full-batch GCN training on graph partitions extended by subgraph
approximation (arXiv 2012.04930), as CUDA kernels for sm_100a behind a C-ABI
library.  ``gcnsa`` is the ctypes binding; ``build`` compiles the library."""
from . import build, gcnsa  # noqa: F401
