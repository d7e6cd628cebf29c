"""B200-native hot path of TPI-LLM (tensor-parallel batch-1 Llama decoding with a
sliding-window weight scheduler).  See include/tpi.h for the C ABI; this package
is a thin ctypes binding over the in-tree CUDA library libtpi.so."""
from .binding import *  # noqa: F401,F403
from .binding import Session, TpiConfig, TpiError, lib, make_config  # noqa: F401
