"""MoR analyse-and-quantise hot path for B200 (sm_100a).

The package holds four things and nothing else:

* ``csrc/``      hand-written CUDA kernels and the C-ABI library ``libmor_b200.so``
* ``binding``    a thin ctypes binding with the same names as the C entry points
* ``workloads``  seeded synthetic input generators (no arithmetic of the method)
* ``sharded``    the two scalar exchanges a row-sharded tensor needs (torch.distributed)

Importing the package does not load the CUDA library; ``binding`` loads it on first
use and raises if it has not been built.
"""

__all__ = ["binding", "workloads", "sharded"]
