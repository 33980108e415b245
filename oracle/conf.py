"""numpy front-end of the oracle's trace-confidence functions (test infrastructure only)."""
import ctypes as C

import numpy as np

from . import _dtype_code, _p, _same_dtype, lib


def token_confidence(hidden, W, rows=None, inv_temp: float = 1.0):
    """H_t = -sum_v log P_t(v), float64 per evaluated row."""
    hidden = np.ascontiguousarray(hidden)
    code = _dtype_code(hidden)
    (W,) = _same_dtype(code, W)
    V, d = W.shape
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
    else:
        n = hidden.shape[0]
    out = np.empty(n, dtype=np.float64)
    rc = lib().oracle_token_confidence(_p(hidden), _p(W), C.c_int(code), _p(rows), C.c_int64(n), C.c_int(d), C.c_int(V),
                                       C.c_double(inv_temp), _p(out))
    if rc != 0:
        raise MemoryError("oracle_token_confidence could not allocate its scratch")
    return out


def trace_confidence(H, cu_seqlens, window: int = 2048, mode: int = 0):
    H = np.ascontiguousarray(H, dtype=np.float64)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int64)
    S = cu.shape[0] - 1
    out = np.empty(S, dtype=np.float64)
    lib().oracle_trace_confidence(_p(H), _p(cu), C.c_int64(S), C.c_int(window), C.c_int(mode), _p(out))
    return out
