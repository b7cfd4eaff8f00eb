"""B200 (sm_100a) implementation of SABlock's prefill-time KV-cache compression pass.

The product is the C-ABI library built from csrc/ (declared in include/sablock.h);
`binding` marshals torch tensors into it.  Importing the package does not load CUDA.
"""
from . import binding, diagnostics, modes  # noqa: F401
from .build import build  # noqa: F401
