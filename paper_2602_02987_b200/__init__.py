"""B200-native many-replication simulator of the gate-and-route LLM-inference queueing network.

`binding.QSim` is a thin ctypes front end of the C-ABI library `libqsim.so` (include/qsim.h): it only
marshals arguments; every simulation step runs in the CUDA kernels.  PyTorch supplies device memory
(the workspace tensor) and the stream.  There is no CPU fallback: without the built library or without
a CUDA device the calls raise.
"""
from .binding import QSim, QSimCTMC, QSimError, load_library, simulate_host, simulate_static, simulate_waves  # noqa: F401
from .build import build_library  # noqa: F401
