"""B200-native 8-bit decentralized training step (arXiv 2111.09389).

`api` binds the C ABI of liblpdt.so one to one; `step.TrainStep` strings the
calls into one whole training step of all simulated nodes; `workloads` holds the
seeded synthetic inputs.  The CUDA library is the only compute path.
"""
from . import workloads  # noqa: F401

__all__ = ["api", "step", "workloads", "build"]
