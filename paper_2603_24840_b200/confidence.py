"""ctypes binding of the trace-confidence calls (marshalling only)."""
import ctypes as C

from . import binding as B

_ready = False


def _lib():
    global _ready
    lib = B.load_library()
    if not _ready:
        lib.arrol_token_logprob_conf.restype = C.c_int
        lib.arrol_token_logprob_conf.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                                 C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                                 C.c_void_p, C.c_size_t, C.c_void_p]
        lib.arrol_trace_confidence.restype = C.c_int
        lib.arrol_trace_confidence.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                               C.c_int32, C.c_void_p, C.c_void_p]
        _ready = True
    return lib


def arrol_token_logprob_conf(ctx: B.Context, hidden, W_vocab, targets, T_max: int, d: int, V: int, logp, token_conf,
                             workspace, lse=None, d_T=None, inv_temperature: float = 1.0, stream=None):
    B._check(_lib().arrol_token_logprob_conf(ctx.handle, B._ptr(hidden), B._ptr(W_vocab), B._ptr(targets), int(T_max),
                                             B._ptr(d_T), int(d), int(V), float(inv_temperature), B._ptr(logp),
                                             B._ptr(lse), B._ptr(token_conf), B._ptr(workspace),
                                             0 if workspace is None else workspace.numel() * workspace.element_size(),
                                             B._stream(stream)), "arrol_token_logprob_conf")


def arrol_trace_confidence(ctx: B.Context, token_conf, cu_seqlens, d_num, S_max: int, trace_conf, window: int = 2048,
                           mode: int = 0, stream=None):
    B._check(_lib().arrol_trace_confidence(ctx.handle, B._ptr(token_conf), B._ptr(cu_seqlens), B._ptr(d_num), int(S_max),
                                           int(window), int(mode), B._ptr(trace_conf), B._stream(stream)),
             "arrol_trace_confidence")
