"""ctypes binding of libarrol.so: argument marshalling only, same names as the C ABI (include/arrol.h).

torch supplies device memory and the current stream; every step of the path runs in the library's CUDA
kernels.  There is no fallback: if the library is missing or no sm_100 device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libarrol.so")

ARROL_F32, ARROL_BF16 = 0, 1
DEV_CAPACITY, DEV_BAD_TARGET, DEV_WAIT_EXPIRED = 1, 2, 4

EXPORTS = [
    "arrol_version", "arrol_status_string", "arrol_create", "arrol_destroy", "arrol_poll_status",
    "arrol_calib_counts", "arrol_build_q_lut", "arrol_score_partial", "arrol_select", "arrol_compact",
    "arrol_token_logprob_workspace", "arrol_token_logprob", "arrol_prune_rebatch_host", "arrol_launch_count",
    "arrol_score_partial_static",
    "arrol_calib_state_bytes", "arrol_calib_layout", "arrol_calib_init", "arrol_calib_update", "arrol_calib_q_lut",
    "arrol_calib_delta", "arrol_select_stochastic",
    "arrol_policy_loss", "arrol_lm_head_backward_workspace", "arrol_lm_head_backward", "arrol_rank_vote",
    "arrol_head_grad_workspace", "arrol_head_grad", "arrol_token_logprob_conf", "arrol_trace_confidence",
    "arrol_prune_step", "arrol_token_logprob_splits", "arrol_token_logprob_form", "arrol_test_hook", "arrol_set_source_rows",
    "arrol_token_logprob_gathered", "arrol_token_logprob_gathered_workspace",
]


class ArrolError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, status_string(code), code))


class _Head(C.Structure):
    _fields_ = [("d", C.c_int32), ("h", C.c_int32), ("dtype", C.c_int32), ("reserved", C.c_int32),
                ("W1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p), ("b2", C.c_void_p)]


class _Calib(C.Structure):
    _fields_ = [("B", C.c_int32), ("reserved", C.c_int32), ("q_lut", C.c_void_p)]


class _HostStep(C.Structure):
    _fields_ = [("P", C.c_int32), ("G", C.c_int32), ("K", C.c_int32), ("cutoff", C.c_int32),
                ("d", C.c_int32), ("V", C.c_int32), ("ddof", C.c_int32), ("reserved", C.c_int32),
                ("rho", C.c_double), ("eps", C.c_float), ("inv_temperature", C.c_float),
                ("T_src", C.c_int64), ("dst_capacity_tokens", C.c_int64),
                ("h_hidden", C.c_void_p), ("h_src_tokens", C.c_void_p), ("h_lengths", C.c_void_p),
                ("h_src_tok_off", C.c_void_p), ("h_rewards", C.c_void_p),
                ("head", _Head), ("calib", _Calib), ("W_vocab", C.c_void_p),
                ("d_hidden", C.c_void_p), ("d_src_tokens", C.c_void_p), ("d_lengths", C.c_void_p),
                ("d_src_tok_off", C.c_void_p), ("d_row_index", C.c_void_p), ("d_rewards", C.c_void_p),
                ("d_score", C.c_void_p), ("d_prob", C.c_void_p), ("d_q", C.c_void_p), ("d_keep", C.c_void_p),
                ("d_survivor_idx", C.c_void_p), ("d_cu_seqlens", C.c_void_p), ("d_adv", C.c_void_p),
                ("d_num", C.c_void_p), ("d_dst_tokens", C.c_void_p), ("d_dst_rows", C.c_void_p),
                ("d_logp", C.c_void_p), ("d_workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("h_logp", C.c_void_p), ("h_adv", C.c_void_p), ("h_cu_seqlens", C.c_void_p),
                ("h_survivor_idx", C.c_void_p), ("h_num", C.c_void_p)]


class _PruneStep(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("row_stride_elems", C.c_int64), ("row_index", C.c_void_p), ("head", _Head),
                ("calib", _Calib), ("score", C.c_void_p), ("prob", C.c_void_p), ("q", C.c_void_p), ("bin", C.c_void_p),
                ("P", C.c_int32), ("G", C.c_int32), ("K", C.c_int32), ("ddof", C.c_int32), ("rho", C.c_double),
                ("keep", C.c_void_p), ("lengths", C.c_void_p), ("src_tok_off", C.c_void_p), ("src_tokens", C.c_void_p),
                ("src_rows", C.c_void_p), ("rewards", C.c_void_p), ("dst_capacity_tokens", C.c_int64),
                ("row_bytes", C.c_int32), ("eps", C.c_float), ("dst_tokens", C.c_void_p), ("dst_rows", C.c_void_p),
                ("cu_seqlens", C.c_void_p), ("survivor_idx", C.c_void_p), ("adv", C.c_void_p), ("tok_adv", C.c_void_p),
                ("tok_seq", C.c_void_p), ("d_num", C.c_void_p)]


_lib = None


def load_library():
    """Loads libarrol.so; raises if it has not been built (python -m paper_2603_24840_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("%s not found: build it with `python paper_2603_24840_b200/build.py` "
                                "(there is no CPU or PyTorch fallback)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    lib.arrol_version.restype = C.c_int
    lib.arrol_status_string.restype = C.c_char_p
    lib.arrol_status_string.argtypes = [C.c_int]
    lib.arrol_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.arrol_destroy.argtypes = [C.c_void_p]
    lib.arrol_poll_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint32)]
    lib.arrol_calib_counts.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]
    lib.arrol_build_q_lut.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_double, C.c_void_p]
    lib.arrol_score_partial.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                        C.POINTER(_Head), C.POINTER(_Calib), C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
    lib.arrol_select.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_double, C.c_int32,
                                 C.c_void_p, C.c_void_p]
    lib.arrol_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                  C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_float, C.c_int32, C.c_int64,
                                  C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_void_p]
    lib.arrol_token_logprob_workspace.restype = C.c_size_t
    lib.arrol_token_logprob_workspace.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32]
    lib.arrol_token_logprob.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                        C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_size_t, C.c_void_p]
    lib.arrol_token_logprob_gathered.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int32,
                                                 C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                                 C.c_void_p]
    lib.arrol_prune_rebatch_host.argtypes = [C.c_void_p, C.POINTER(_HostStep), C.c_void_p]
    lib.arrol_prune_rebatch_host.restype = C.c_int
    lib.arrol_score_partial_static.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.POINTER(_Head),
                                               C.POINTER(_Calib), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p]
    lib.arrol_score_partial_static.restype = C.c_int
    lib.arrol_prune_step.argtypes = [C.c_void_p, C.POINTER(_PruneStep), C.c_void_p]
    lib.arrol_prune_step.restype = C.c_int
    lib.arrol_launch_count.argtypes = [C.c_void_p]
    lib.arrol_launch_count.restype = C.c_int64
    for fn in ("arrol_create", "arrol_destroy", "arrol_poll_status", "arrol_calib_counts", "arrol_build_q_lut",
               "arrol_score_partial", "arrol_select", "arrol_compact", "arrol_token_logprob"):
        getattr(lib, fn).restype = C.c_int
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().arrol_status_string(int(code)).decode()


def arrol_version() -> int:
    return int(load_library().arrol_version())


def _check(code: int, where: str):
    if code != 0:
        raise ArrolError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ARROL_F32
    if t.dtype == torch.bfloat16:
        return ARROL_BF16
    raise TypeError("hidden / head tensors are float32 or bfloat16")


class Context:
    """Owns an arrol_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        lib = load_library()
        self._h = C.c_void_p()
        _check(lib.arrol_create(C.byref(self._h), int(device)), "arrol_create")
        self.device = int(device)

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            load_library().arrol_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def handle(self):
        return self._h


def arrol_poll_status(ctx: Context, stream=None, raise_on_error: bool = True) -> int:
    bits = C.c_uint32(0)
    rc = load_library().arrol_poll_status(ctx.handle, _stream(stream), C.byref(bits))
    if rc != 0 and raise_on_error:
        raise ArrolError(rc, "arrol_poll_status (device bits = %d)" % bits.value)
    return int(bits.value)


def arrol_calib_counts(sprime, y, B: int):
    """Host helper: histogram counts of historical scores per bin (numpy in, numpy out)."""
    import numpy as np
    sprime = np.ascontiguousarray(sprime, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.uint8)
    cpos = np.empty(B, dtype=np.int64)
    cneg = np.empty(B, dtype=np.int64)
    _check(load_library().arrol_calib_counts(sprime.ctypes.data, y.ctypes.data, sprime.shape[0], int(B),
                                             cpos.ctypes.data, cneg.ctypes.data), "arrol_calib_counts")
    return cpos, cneg


def arrol_build_q_lut(cpos, cneg, alpha: float = 1.0):
    """Host helper: posterior per bin as float32 numpy [B]."""
    import numpy as np
    cpos = np.ascontiguousarray(cpos, dtype=np.int64)
    cneg = np.ascontiguousarray(cneg, dtype=np.int64)
    B = cpos.shape[0]
    q = np.empty(B, dtype=np.float32)
    _check(load_library().arrol_build_q_lut(cpos.ctypes.data, cneg.ctypes.data, int(B), float(alpha),
                                            q.ctypes.data), "arrol_build_q_lut")
    return q


def arrol_score_partial(ctx: Context, hidden: torch.Tensor, head: dict, N: int, score: torch.Tensor,
                        prob: torch.Tensor, q: torch.Tensor, bin: Optional[torch.Tensor] = None,
                        row_index: Optional[torch.Tensor] = None, q_lut: Optional[torch.Tensor] = None,
                        row_stride: Optional[int] = None, stream=None):
    """head = {"W1", "b1", "w2", "b2", "h"} (device tensors or None).  Outputs are written in place."""
    hs = _Head()
    hs.d = hidden.shape[-1]
    hs.h = int(head.get("h", 0))
    hs.dtype = _dtype_code(hidden)
    for name in ("W1", "b1", "w2", "b2"):
        t = head.get(name)
        if t is not None and t.dtype != hidden.dtype:
            raise TypeError("head tensors share the hidden dtype")
        setattr(hs, name, None if t is None else t.data_ptr())
    cs = _Calib()
    cs.B = 0 if q_lut is None else q_lut.shape[0]
    cs.q_lut = None if q_lut is None else q_lut.data_ptr()
    stride = hidden.stride(-2) if row_stride is None else int(row_stride)
    _check(load_library().arrol_score_partial(ctx.handle, _ptr(hidden), stride, _ptr(row_index), int(N),
                                              C.byref(hs), C.byref(cs), _ptr(score), _ptr(prob), _ptr(bin),
                                              _ptr(q), _stream(stream)), "arrol_score_partial")


def arrol_select(ctx: Context, q: torch.Tensor, P: int, G: int, K: int, rho: float, keep: torch.Tensor,
                 mode: int = 0, stream=None):
    _check(load_library().arrol_select(ctx.handle, _ptr(q), int(P), int(G), int(K), float(rho), int(mode),
                                       _ptr(keep), _stream(stream)), "arrol_select")


def arrol_compact(ctx: Context, keep, lengths, src_tok_off, N: int, G: int, rewards, dst_capacity_tokens: int,
                  cu_seqlens, survivor_idx, adv, d_num, src_tokens=None, dst_tokens=None, src_rows=None,
                  dst_rows=None, row_bytes: int = 0, tok_adv=None, tok_seq=None, eps: float = 1e-6, ddof: int = 0,
                  stream=None):
    _check(load_library().arrol_compact(ctx.handle, _ptr(keep), _ptr(lengths), _ptr(src_tok_off), int(N), int(G),
                                        _ptr(src_tokens), _ptr(src_rows), int(row_bytes), _ptr(rewards),
                                        float(eps), int(ddof), int(dst_capacity_tokens), _ptr(dst_tokens),
                                        _ptr(dst_rows), _ptr(cu_seqlens), _ptr(survivor_idx), _ptr(adv),
                                        _ptr(tok_adv), _ptr(tok_seq), _ptr(d_num), _stream(stream)),
           "arrol_compact")


def arrol_token_logprob_workspace(ctx: Context, T_max: int, d: int, V: int) -> int:
    return int(load_library().arrol_token_logprob_workspace(ctx.handle, int(T_max), int(d), int(V)))


def arrol_token_logprob_form(ctx: Context, T_max: int, d: int, V: int) -> int:
    """2 = the kernel runs as pairs of blocks on 256-row tiles for these sizes, 1 = one block per 128-row tile."""
    lib = load_library()
    lib.arrol_token_logprob_form.restype = C.c_int32
    lib.arrol_token_logprob_form.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32]
    return int(lib.arrol_token_logprob_form(ctx.handle, int(T_max), int(d), int(V)))


def arrol_token_logprob_splits(ctx: Context, T_max: int, d: int, V: int) -> int:
    lib = load_library()
    lib.arrol_token_logprob_splits.restype = C.c_int32
    lib.arrol_token_logprob_splits.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32]
    return int(lib.arrol_token_logprob_splits(ctx.handle, int(T_max), int(d), int(V)))


def arrol_token_logprob(ctx: Context, hidden, W_vocab, targets, T_max: int, d: int, V: int, logp, workspace,
                        lse=None, d_T=None, inv_temperature: float = 1.0, stream=None):
    _check(load_library().arrol_token_logprob(ctx.handle, _ptr(hidden), _ptr(W_vocab), _ptr(targets), int(T_max),
                                              _ptr(d_T), int(d), int(V), float(inv_temperature), _ptr(logp),
                                              _ptr(lse), _ptr(workspace),
                                              0 if workspace is None else workspace.numel() * workspace.element_size(),
                                              _stream(stream)), "arrol_token_logprob")


def arrol_token_logprob_gathered_workspace(ctx: Context, S_max: int, T_max: int, d: int, V: int) -> int:
    lib = load_library()
    lib.arrol_token_logprob_gathered_workspace.restype = C.c_size_t
    lib.arrol_token_logprob_gathered_workspace.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_int32, C.c_int32]
    return int(lib.arrol_token_logprob_gathered_workspace(ctx.handle, int(S_max), int(T_max), int(d), int(V)))


def arrol_token_logprob_gathered(ctx: Context, src_rows, W_vocab, targets, cu_seqlens, survivor_idx, src_tok_off, d_num,
                                 S_max: int, T_max: int, d: int, V: int, logp, workspace, lse=None,
                                 inv_temperature: float = 1.0, source_rows: Optional[int] = None, stream=None):
    """Log-probs of the packed survivor tokens with the hidden rows read from the pre-prune buffer `src_rows`."""
    rows = src_rows.shape[0] if source_rows is None else int(source_rows)
    _check(load_library().arrol_token_logprob_gathered(
        ctx.handle, _ptr(src_rows), rows, _ptr(W_vocab), _ptr(targets), _ptr(cu_seqlens), _ptr(survivor_idx),
        _ptr(src_tok_off), _ptr(d_num), int(S_max), int(T_max), int(d), int(V), float(inv_temperature), _ptr(logp),
        _ptr(lse), _ptr(workspace), 0 if workspace is None else workspace.numel() * workspace.element_size(),
        _stream(stream)), "arrol_token_logprob_gathered")


HOOK_SPIN_LIMIT, HOOK_MUTE_LOGPROB_PRODUCER, HOOK_LOGPROB_TIMING_BUFFER, HOOK_LOGPROB_TIMING_ITEMS, HOOK_LOGPROB_PAIR, HOOK_LOGPROB_SPLITS = 1, 2, 3, 4, 5, 6


def arrol_test_hook(ctx: Context, key: int, value: int):
    """Test hook: bounds the log-prob kernel's pipeline waits / silences its producer (see include/arrol.h)."""
    lib = load_library()
    lib.arrol_test_hook.argtypes = [C.c_void_p, C.c_int32, C.c_int64]
    _check(lib.arrol_test_hook(ctx.handle, int(key), int(value)), "arrol_test_hook")


def arrol_set_source_rows(ctx: Context, source_rows: int):
    """Switches on (source_rows > 0) or off (0) the device-side range checks of row_index / src_tok_off + lengths."""
    lib = load_library()
    lib.arrol_set_source_rows.argtypes = [C.c_void_p, C.c_int64]
    _check(lib.arrol_set_source_rows(ctx.handle, int(source_rows)), "arrol_set_source_rows")


def arrol_launch_count(ctx: Context) -> int:
    return int(load_library().arrol_launch_count(ctx.handle))


def _fill_head(hs: _Head, hidden_dtype_code: int, d: int, head: dict):
    hs.d = int(d)
    hs.h = int(head.get("h", 0))
    hs.dtype = hidden_dtype_code
    for name in ("W1", "b1", "w2", "b2"):
        t = head.get(name)
        setattr(hs, name, None if t is None else t.data_ptr())


def make_host_step(scalars: dict, head: dict, q_lut: Optional[torch.Tensor], tensors: dict) -> _HostStep:
    """Builds the argument block of arrol_prune_rebatch_host.  `scalars`: P, G, K, cutoff, d, V, rho, eps, ddof,
    inv_temperature, T_src, dst_capacity_tokens.  `tensors`: every h_* (CPU tensors) and d_* (CUDA tensors) field
    plus W_vocab.  The caller keeps the tensors alive while the block is in use."""
    st = _HostStep()
    for k, v in scalars.items():
        setattr(st, k, v)
    _fill_head(st.head, ARROL_BF16, scalars["d"], head)
    st.calib.B = 0 if q_lut is None else q_lut.shape[0]
    st.calib.q_lut = None if q_lut is None else q_lut.data_ptr()
    for k, t in tensors.items():
        if k.startswith("h_") and t.is_cuda:
            raise ValueError("%s must be a host tensor" % k)
        if (k.startswith("d_") or k == "W_vocab") and not t.is_cuda:
            raise ValueError("%s must be a device tensor" % k)
        setattr(st, k, t.data_ptr())
    st.workspace_bytes = tensors["d_workspace"].numel() * tensors["d_workspace"].element_size()
    return st


def arrol_prune_rebatch_host(ctx: Context, step: _HostStep, stream=None):
    _check(load_library().arrol_prune_rebatch_host(ctx.handle, C.byref(step), _stream(stream)),
           "arrol_prune_rebatch_host")


def arrol_score_partial_static(hidden: torch.Tensor, head: dict, N: int, score: torch.Tensor, prob: torch.Tensor,
                               q: torch.Tensor, bin: Optional[torch.Tensor] = None,
                               row_index: Optional[torch.Tensor] = None, q_lut: Optional[torch.Tensor] = None,
                               row_stride: Optional[int] = None, stream=None):
    """MLP-head scoring for callers that may not allocate device memory (a frozen memory plan, a host
    application that owns the device heap, a latency-critical loop): no context, no allocation; the scratch is
    a fixed 128 KiB array inside the library.  Limits: MLP head only, N <= 4096, h <= 512.  Runs on the current
    device; calls that overlap on one GPU race on the shared scratch.  The first call per device does a one-time
    address look-up and should come before any stream capture."""
    hs = _Head()
    _fill_head(hs, _dtype_code(hidden), hidden.shape[-1], head)
    cs = _Calib()
    cs.B = 0 if q_lut is None else q_lut.shape[0]
    cs.q_lut = None if q_lut is None else q_lut.data_ptr()
    stride = hidden.stride(-2) if row_stride is None else int(row_stride)
    _check(load_library().arrol_score_partial_static(_ptr(hidden), stride, _ptr(row_index), int(N), C.byref(hs),
                                                     C.byref(cs), _ptr(score), _ptr(prob), _ptr(bin), _ptr(q),
                                                     _stream(stream)), "arrol_score_partial_static")


def make_prune_step(hidden: torch.Tensor, head: dict, q_lut: Optional[torch.Tensor], scalars: dict, tensors: dict,
                    row_stride: Optional[int] = None) -> _PruneStep:
    """Argument block of arrol_prune_step.  scalars: P, G, K, rho, eps, ddof, dst_capacity_tokens, row_bytes;
    tensors: the device tensors by field name (missing / None = NULL).  The caller keeps the tensors alive."""
    a = _PruneStep()
    a.hidden = hidden.data_ptr()
    a.row_stride_elems = hidden.stride(-2) if row_stride is None else int(row_stride)
    _fill_head(a.head, _dtype_code(hidden), hidden.shape[-1], head)
    a.calib.B = 0 if q_lut is None else q_lut.shape[0]
    a.calib.q_lut = None if q_lut is None else q_lut.data_ptr()
    for k, v in scalars.items():
        setattr(a, k, v)
    for k, t in tensors.items():
        setattr(a, k, None if t is None else t.data_ptr())
    return a


def arrol_prune_step(ctx: Context, args: _PruneStep, stream=None):
    _check(load_library().arrol_prune_step(ctx.handle, C.byref(args), _stream(stream)), "arrol_prune_step")
