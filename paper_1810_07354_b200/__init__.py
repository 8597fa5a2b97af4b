"""SCAR checkpoint-and-recover parameter pass for one B200 (sm_100a).

``libscar.so`` (hand-written CUDA behind a C ABI, see ``include/scar.h``) does
all the work; :mod:`paper_1810_07354_b200.api` is a thin ctypes binding with
the same names.  There is no CPU fallback: calls fail loudly when the library
or a CUDA device is missing.
"""

from .api import (  # noqa: F401
    SCAR_F32,
    SCAR_I32,
    ScarError,
    ScarCheckpoint,
    lib_path,
    load_library,
    exported_symbols,
)
