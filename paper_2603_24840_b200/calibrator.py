"""ctypes binding of the online calibrator and the stochastic pruning rule (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np
import torch

from . import binding as B


class _Survival(C.Structure):
    _fields_ = [("kappa", C.c_double), ("lambda_", C.c_double), ("rho", C.c_double), ("p_min", C.c_double),
                ("p_max", C.c_double)]


def survival(kappa=0.5, lam=0.5, rho=0.5, p_min=0.05, p_max=0.95) -> _Survival:
    return _Survival(kappa, lam, rho, p_min, p_max)


_ready = False


def _lib():
    global _ready
    lib = B.load_library()
    if not _ready:
        lib.arrol_calib_state_bytes.restype = C.c_size_t
        lib.arrol_calib_state_bytes.argtypes = [C.c_int32, C.c_int64]
        lib.arrol_calib_layout.restype = C.c_int
        lib.arrol_calib_layout.argtypes = [C.c_int32, C.c_int64, C.POINTER(C.c_size_t)]
        lib.arrol_calib_init.restype = C.c_int
        lib.arrol_calib_init.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int32, C.c_int64, C.c_double, C.c_void_p]
        lib.arrol_calib_update.restype = C.c_int
        lib.arrol_calib_update.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_int32, C.POINTER(_Survival), C.c_void_p]
        lib.arrol_calib_q_lut.restype = C.c_void_p
        lib.arrol_calib_q_lut.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
        lib.arrol_calib_delta.restype = C.c_void_p
        lib.arrol_calib_delta.argtypes = [C.c_void_p]
        lib.arrol_select_stochastic.restype = C.c_int
        lib.arrol_select_stochastic.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                                C.POINTER(_Survival), C.c_void_p, C.c_double, C.c_void_p, C.c_void_p,
                                                C.c_void_p]
        _ready = True
    return lib


def arrol_calib_state_bytes(n_bins: int, cap: int) -> int:
    return int(_lib().arrol_calib_state_bytes(int(n_bins), int(cap)))


def arrol_calib_layout(n_bins: int, cap: int):
    off = (C.c_size_t * 6)()
    B._check(_lib().arrol_calib_layout(int(n_bins), int(cap), off), "arrol_calib_layout")
    return dict(zip(("cpos", "cneg", "q_lut", "ring_pos", "ring_neg", "total"), (int(v) for v in off)))


class Calibrator:
    """Device-resident calibrator state in a torch-allocated buffer."""

    def __init__(self, ctx: B.Context, n_bins: int = 128, cap: int = 8192, alpha: float = 1.0, device=None):
        self.ctx, self.n_bins, self.cap = ctx, int(n_bins), int(cap)
        nbytes = arrol_calib_state_bytes(n_bins, cap)
        if nbytes == 0:
            raise ValueError("unsupported calibrator shape")
        self.state = torch.empty(nbytes, dtype=torch.uint8, device=device or torch.device("cuda", ctx.device))
        B._check(_lib().arrol_calib_init(ctx.handle, B._ptr(self.state), nbytes, self.n_bins, self.cap, float(alpha),
                                         B._stream()), "arrol_calib_init")
        lay = arrol_calib_layout(n_bins, cap)
        self.layout = lay
        # views into the state (no copies): the table feeds arrol_score_partial, delta feeds arrol_select_stochastic
        self.q_lut = self.state[lay["q_lut"]:lay["q_lut"] + 4 * self.n_bins].view(torch.float32)
        self.delta = self.state[56:64].view(torch.float64)
        assert self.q_lut.data_ptr() == _lib().arrol_calib_q_lut(B._ptr(self.state), self.n_bins, self.cap)
        assert self.delta.data_ptr() == _lib().arrol_calib_delta(B._ptr(self.state))

    def update(self, bins: torch.Tensor, rewards: torch.Tensor, params: _Survival, mask: Optional[torch.Tensor] = None,
               stream=None):
        B._check(_lib().arrol_calib_update(self.ctx.handle, B._ptr(self.state), self.n_bins, self.cap, B._ptr(bins),
                                           B._ptr(rewards), B._ptr(mask), int(bins.shape[0]), C.byref(params),
                                           B._stream(stream)), "arrol_calib_update")

    def snapshot(self):
        """Host copy of the state: counts, rings in oldest-to-newest order, table, delta."""
        raw = self.state.cpu().numpy()
        lay, nb, cap = self.layout, self.n_bins, self.cap
        hdr = raw[:64].view(np.int64)
        head_pos, n_pos, head_neg, n_neg = (int(hdr[i]) for i in (2, 3, 4, 5))
        ring_pos = raw[lay["ring_pos"]:lay["ring_pos"] + 2 * cap].view(np.int16)
        ring_neg = raw[lay["ring_neg"]:lay["ring_neg"] + 2 * cap].view(np.int16)
        return {
            "cpos": raw[lay["cpos"]:lay["cpos"] + 8 * nb].view(np.int64).copy(),
            "cneg": raw[lay["cneg"]:lay["cneg"] + 8 * nb].view(np.int64).copy(),
            "q_lut": raw[lay["q_lut"]:lay["q_lut"] + 4 * nb].view(np.float32).copy(),
            "pos": np.array([ring_pos[(head_pos + i) % cap] for i in range(n_pos)], dtype=np.int64),
            "neg": np.array([ring_neg[(head_neg + i) % cap] for i in range(n_neg)], dtype=np.int64),
            "delta": float(raw[56:64].view(np.float64)[0]),
        }


def arrol_select_stochastic(ctx: B.Context, q: torch.Tensor, u: torch.Tensor, keep: torch.Tensor, params: _Survival,
                            d_delta: Optional[torch.Tensor] = None, delta: float = 0.0,
                            eligible: Optional[torch.Tensor] = None, p_out: Optional[torch.Tensor] = None, stream=None):
    B._check(_lib().arrol_select_stochastic(ctx.handle, B._ptr(q), B._ptr(u), B._ptr(eligible), int(q.shape[0]),
                                            C.byref(params), B._ptr(d_delta), float(delta), B._ptr(keep),
                                            B._ptr(p_out), B._stream(stream)), "arrol_select_stochastic")
