"""ctypes binding of the policy-update calls: clipped objective and lm_head log-prob backward (marshalling only)."""
from __future__ import annotations

import ctypes as C
from typing import Optional

import torch

from . import binding as B

_ready = False


def _lib():
    global _ready
    lib = B.load_library()
    if not _ready:
        lib.arrol_policy_loss.restype = C.c_int
        lib.arrol_policy_loss.argtypes = [C.c_void_p] * 8 + [C.c_int64, C.c_float, C.c_float, C.c_float, C.c_int32,
                                                             C.c_void_p, C.c_void_p, C.c_void_p]
        lib.arrol_lm_head_backward_workspace.restype = C.c_size_t
        lib.arrol_lm_head_backward_workspace.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32]
        lib.arrol_lm_head_backward.restype = C.c_int
        lib.arrol_lm_head_backward.argtypes = [C.c_void_p] * 6 + [C.c_int64, C.c_void_p, C.c_int32, C.c_int32, C.c_float,
                                                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        _ready = True
    return lib


def arrol_policy_loss(ctx: B.Context, logp, logp_old, tok_adv, tok_seq, cu_seqlens, d_num, T_max: int, grad_logp, loss,
                      logp_ref: Optional[torch.Tensor] = None, eps_low: float = 0.2, eps_high: float = 0.2,
                      beta: float = 0.0, agg_mode: int = 0, stream=None):
    B._check(_lib().arrol_policy_loss(ctx.handle, B._ptr(logp), B._ptr(logp_old), B._ptr(logp_ref), B._ptr(tok_adv),
                                      B._ptr(tok_seq), B._ptr(cu_seqlens), B._ptr(d_num), int(T_max), float(eps_low),
                                      float(eps_high), float(beta), int(agg_mode), B._ptr(grad_logp), B._ptr(loss),
                                      B._stream(stream)), "arrol_policy_loss")


def arrol_lm_head_backward_workspace(ctx: B.Context, T_max: int, d: int, V: int) -> int:
    return int(_lib().arrol_lm_head_backward_workspace(ctx.handle, int(T_max), int(d), int(V)))


def arrol_lm_head_backward(ctx: B.Context, hidden, W_vocab, targets, grad_logp, lse, T_max: int, d: int, V: int, dH, dW,
                           workspace, d_T=None, inv_temperature: float = 1.0, stream=None):
    B._check(_lib().arrol_lm_head_backward(ctx.handle, B._ptr(hidden), B._ptr(W_vocab), B._ptr(targets),
                                           B._ptr(grad_logp), B._ptr(lse), int(T_max), B._ptr(d_T), int(d), int(V),
                                           float(inv_temperature), B._ptr(dH), B._ptr(dW), B._ptr(workspace),
                                           0 if workspace is None else workspace.numel() * workspace.element_size(),
                                           B._stream(stream)), "arrol_lm_head_backward")
