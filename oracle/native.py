"""ctypes access to the C++ oracle (oracle/topk_oracle.cpp)."""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        sig = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        for name in ("oracle_topk_stable_sort", "oracle_topk_nth_element"):
            fn = getattr(_lib, name)
            fn.argtypes = sig
            fn.restype = ctypes.c_int
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def max_threads():
    return int(lib().oracle_max_threads())


def _run(name, scores, row_starts, row_lengths, K, num_threads):
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    row_starts = np.ascontiguousarray(row_starts, dtype=np.int32)
    row_lengths = np.ascontiguousarray(row_lengths, dtype=np.int32)
    M = len(row_lengths)
    out_idx = np.empty((M, K), dtype=np.int32)
    out_val = np.empty((M, K), dtype=np.float32)
    used = getattr(lib(), name)(scores.ctypes.data, row_starts.ctypes.data,
                                row_lengths.ctypes.data, M, K, out_idx.ctypes.data,
                                out_val.ctypes.data, num_threads)
    return out_idx, out_val, used


def topk_stable_sort(scores, row_starts, row_lengths, K, num_threads=0):
    """The definition (stable sort per row); returns (idx, val, threads_used)."""
    return _run("oracle_topk_stable_sort", scores, row_starts, row_lengths, K, num_threads)


def topk_nth_element(scores, row_starts, row_lengths, K, num_threads=0):
    """Independent nth_element selector; returns (idx, val, threads_used)."""
    return _run("oracle_topk_nth_element", scores, row_starts, row_lengths, K, num_threads)
