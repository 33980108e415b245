"""numpy front-end of the oracle's quality-head training step (test infrastructure only)."""
import ctypes as C

import numpy as np

from . import _dtype_code, _p, _same_dtype, lib


def head_bce_grad(hidden, y, W1, b1=None, w2=None, b2=None, row_index=None, h: int = 0, mask=None):
    """Binary cross-entropy of the head's logits against the final rewards and its gradient with respect to the
    head's parameters.  Returns (loss, dict of float64 gradients)."""
    hidden = np.ascontiguousarray(hidden)
    code = _dtype_code(hidden)
    W1, b1, w2, b2 = _same_dtype(code, W1, b1, w2, b2)
    d = hidden.shape[-1]
    if row_index is not None:
        row_index = np.ascontiguousarray(row_index, dtype=np.int64)
        N = row_index.shape[0]
    else:
        N = hidden.shape[0]
    y = np.ascontiguousarray(y, dtype=np.uint8)
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
    hh = max(h, 1)
    out = {"W1": np.empty((hh, d) if h else (d,), np.float64), "b1": np.empty(hh, np.float64),
           "w2": np.empty(hh, np.float64), "b2": np.empty(1, np.float64)}
    loss = C.c_double(0.0)
    rc = lib().oracle_head_bce_grad(_p(hidden), C.c_int(code), C.c_int64(d), _p(row_index), C.c_int(N), C.c_int(d),
                                    C.c_int(h), _p(W1), _p(b1), _p(w2), _p(b2), _p(y), _p(mask), C.byref(loss),
                                    _p(out["W1"]), _p(out["b1"]), _p(out["w2"]), _p(out["b2"]))
    if rc != 0:
        raise MemoryError("oracle_head_bce_grad could not allocate its scratch")
    if h == 0:
        out.pop("w2")
        out.pop("b2")
    return float(loss.value), out
