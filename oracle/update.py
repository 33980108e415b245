"""numpy front-end of the oracle's policy-update functions (test infrastructure only)."""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import _dtype_code, _p, _same_dtype, lib


def policy_loss(logp, logp_old, tok_adv, cu_seqlens, logp_ref=None, eps_low=0.2, eps_high=0.2, beta=0.0, agg_mode=0):
    """Clipped GRPO (agg_mode 0) / DAPO (agg_mode 1) loss on the packed survivors.  Returns (loss, grad wrt logp)."""
    f64 = lambda a: None if a is None else np.ascontiguousarray(a, dtype=np.float64)
    logp, logp_old, logp_ref, tok_adv = f64(logp), f64(logp_old), f64(logp_ref), f64(tok_adv)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int64)
    S = cu.shape[0] - 1
    grad = np.zeros(int(cu[S]), dtype=np.float64)
    loss = C.c_double(0.0)
    lib().oracle_policy_loss(_p(logp), _p(logp_old), _p(logp_ref), _p(tok_adv), _p(cu), C.c_int64(S),
                             C.c_double(eps_low), C.c_double(eps_high), C.c_double(beta), C.c_int(agg_mode),
                             C.byref(loss), _p(grad))
    return float(loss.value), grad


def lm_head_backward(hidden, W, targets, g, inv_temp: float = 1.0):
    """Returns (dH [T,d], dW [V,d]) in float64."""
    hidden = np.ascontiguousarray(hidden)
    code = _dtype_code(hidden)
    (W,) = _same_dtype(code, W)
    targets = np.ascontiguousarray(targets, dtype=np.int32)
    g = np.ascontiguousarray(g, dtype=np.float64)
    T, d = hidden.shape
    V = W.shape[0]
    dH = np.empty((T, d), dtype=np.float64)
    dW = np.empty((V, d), dtype=np.float64)
    rc = lib().oracle_lm_head_backward(_p(hidden), _p(W), C.c_int(code), _p(targets), _p(g), C.c_int64(T), C.c_int(d),
                                       C.c_int(V), C.c_double(inv_temp), _p(dH), _p(dW))
    if rc != 0:
        raise MemoryError("oracle_lm_head_backward could not allocate its scratch")
    return dH, dW
