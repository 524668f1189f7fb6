"""Helpers that only tests use."""
import ctypes as C
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "early_producer.cu")
_LIB = os.path.join(_HERE, "libearly_producer.so")


def early_producer_lib():
    """The producer kernel of early_producer.cu, compiled for sm_100a next to its source."""
    if not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-shared",
                               "-Xcompiler", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    L = C.CDLL(_LIB)
    L.early_producer.restype = C.c_int
    L.early_producer.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_longlong, C.c_void_p]
    return L
