"""B200-native multi-coil SENSE data-consistency step (GLEAM, arXiv 2207.08393, Eq. 3) and its
vector-Jacobian product.  The arithmetic lives in the CUDA library ``libgleam_dc.so`` (C ABI in
``include/gleam.h``); this package is the argument-marshalling binding plus the seeded synthetic
workload generators."""
from . import workloads  # noqa: F401

__all__ = ["workloads"]
