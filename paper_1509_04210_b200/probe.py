"""ctypes access to ``librudra_probe.so``, the benchmark's bandwidth probe (a library of its own,
outside the parameter-server interface).  Marshalling only."""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        path = _build.PROBE_LIB_PATH
        if not os.path.exists(path) or _build.needs_build(path):
            try:
                _build.build_probe()
            except Exception as exc:
                if not os.path.exists(path):
                    raise ImportError("librudra_probe.so is missing and could not be built: %r" % (exc,)) from exc
        L = C.CDLL(path)
        L.rudra_stream_probe.restype = C.c_int
        L.rudra_stream_probe.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint32, C.c_uint64, C.c_void_p]
        _lib = L
    return _lib


def _table(xs):
    return (C.c_void_p * len(xs))(*[x if isinstance(x, int) else x.data_ptr() for x in xs])


def stream_probe(srcs_dev, dsts_dev, nfloats, stream=None):
    """One launch that only reads srcs_dev and writes dsts_dev (their contents are lost)."""
    handle = stream.cuda_stream if hasattr(stream, "cuda_stream") else stream
    code = lib().rudra_stream_probe(_table(srcs_dev) if srcs_dev else None, len(srcs_dev),
                                    _table(dsts_dev) if dsts_dev else None, len(dsts_dev), int(nfloats), handle)
    if code < 0:
        raise RuntimeError("rudra_stream_probe refused its arguments or the launch failed (%d)" % code)
    return code
