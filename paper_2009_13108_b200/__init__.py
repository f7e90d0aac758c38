"""B200 (sm_100a) implementation of the NITI integer-training hot path.

``Niti`` is a thin ctypes binding of the C-ABI library declared in ``include/niti.h`` (argument
marshalling only; every step runs in the CUDA kernels).  ``NitiTrainer`` strings the calls of one
training step (Algorithm 1 of the paper) together for a feed-forward net.  There is no CPU
fallback: importing works without a GPU, but constructing ``Niti`` requires the built library
and a CUDA device.
"""
from .api import Niti, NitiError, dist_reducer, library_path  # noqa: F401
from .trainer import NitiTrainer  # noqa: F401
