"""B200-native dual-basis Power-of-Two linear kernels (GoQuant inner product).

`paper_2605_26092_b200.goq` is a thin ctypes binding over libgoq.so (include/goq.h): it marshals
arguments only; every step of the path runs in the CUDA kernels. There is no CPU fallback:
loading fails loudly if the library has not been built.
"""
from . import goq  # noqa: F401
