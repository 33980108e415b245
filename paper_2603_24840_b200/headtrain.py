"""ctypes binding of the quality-head training step (marshalling only)."""
import ctypes as C
from typing import Optional

import torch

from . import binding as B

_ready = False


def _lib():
    global _ready
    lib = B.load_library()
    if not _ready:
        lib.arrol_head_grad_workspace.restype = C.c_size_t
        lib.arrol_head_grad_workspace.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32]
        lib.arrol_head_grad.restype = C.c_int
        lib.arrol_head_grad.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.POINTER(B._Head)] + \
            [C.c_void_p] * 8 + [C.c_size_t, C.c_void_p]
        _ready = True
    return lib


def arrol_head_grad_workspace(ctx: B.Context, N: int, d: int, h: int) -> int:
    return int(_lib().arrol_head_grad_workspace(ctx.handle, int(N), int(d), int(h)))


def arrol_head_grad(ctx: B.Context, hidden: torch.Tensor, head: dict, N: int, rewards, grads: dict, loss, workspace,
                    row_index: Optional[torch.Tensor] = None, mask: Optional[torch.Tensor] = None, stream=None):
    """grads = {"W1", "b1"[, "w2", "b2"]} float32 device tensors, overwritten; loss = float64 device tensor [1]."""
    hs = B._Head()
    B._fill_head(hs, B._dtype_code(hidden), hidden.shape[-1], head)
    B._check(_lib().arrol_head_grad(ctx.handle, B._ptr(hidden), hidden.stride(-2), B._ptr(row_index), int(N),
                                    C.byref(hs), B._ptr(rewards), B._ptr(mask), B._ptr(grads["W1"]), B._ptr(grads["b1"]),
                                    B._ptr(grads.get("w2")), B._ptr(grads.get("b2")), B._ptr(loss), B._ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    B._stream(stream)), "arrol_head_grad")
