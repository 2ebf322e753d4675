"""B200-native hot path of DP-SGD with ghost clipping (sm_100a CUDA behind a C ABI).

`workloads` draws seeded synthetic inputs (numpy only).  `binding` is the thin
ctypes layer over the shared library built from `csrc/`; it raises if that
library is missing -- there is no CPU fallback.
"""
__version__ = "0.1.0"
