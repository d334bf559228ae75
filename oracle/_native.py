"""Build and load the oracle's small C file (TEST INFRASTRUCTURE ONLY).

``ef_arith.c`` is compiled with plain gcc, without fast-math and without contraction, so the
only fused operations are the explicit ``fmaf`` calls.
"""
import ctypes
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ef_arith.c")
_LIB = os.path.join(_HERE, "libef_arith.so")
_lib = None


def build(force=False):
    """Compile ef_arith.c into libef_arith.so next to it (no-op when up to date)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-ffp-contract=off",
           "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_accumulate.argtypes = [ctypes.c_float, ctypes.c_void_p, ctypes.c_int,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64]
        L.orc_accumulate.restype = None
        L.orc_apply.argtypes = [ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p,
                                ctypes.c_uint64]
        L.orc_apply.restype = None
        _lib = L
    return _lib
