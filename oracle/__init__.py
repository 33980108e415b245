"""numpy front-end of the CPU oracle (test infrastructure only).

Compiles ``arrol_oracle.c`` with gcc on first use and calls it through ctypes.
Nothing here is imported by the CUDA library or its Python binding; only the
tests, the smoke check and the bench's CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "arrol_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

F32, BF16, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle (plain C, -O2, no fast-math, no FMA contraction, OpenMP over independent units)."""
    srcs = sorted(os.path.join(_HERE, f) for f in os.listdir(_HERE) if f.endswith(".c"))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(s) for s in srcs):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC"] +
                              srcs + ["-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_num_threads.restype = C.c_int
        _lib.oracle_bin_index.restype = C.c_int
        _lib.oracle_bin_index.argtypes = [C.c_double, C.c_int]
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("oracle arrays are float32, float64 or uint16 (bf16 bits), got %s" % a.dtype)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _same_dtype(code, *arrs):
    out = []
    for a in arrs:
        if a is None:
            out.append(None)
            continue
        a = np.ascontiguousarray(a)
        if _dtype_code(a) != code:
            raise TypeError("all floating inputs of one call share a dtype")
        out.append(a)
    return out


def head_score(hidden, W1, b1=None, w2=None, b2=None, row_index=None, h: int = 0, row_stride=None):
    """Quality-head score per rollout, float64 [N] (Section 4.2)."""
    hidden = np.ascontiguousarray(hidden)
    code = _dtype_code(hidden)
    W1, b1, w2, b2 = _same_dtype(code, W1, b1, w2, b2)
    d = hidden.shape[-1]
    stride = d if row_stride is None else int(row_stride)
    if row_index is not None:
        row_index = np.ascontiguousarray(row_index, dtype=np.int64)
        N = row_index.shape[0]
    else:
        N = hidden.reshape(-1, d).shape[0]
    score = np.empty(N, dtype=np.float64)
    rc = lib().oracle_head_score(_p(hidden), C.c_int(code), C.c_int64(stride), _p(row_index), C.c_int(N),
                                 C.c_int(d), C.c_int(h), _p(W1), _p(b1), _p(w2), _p(b2), _p(score))
    if rc != 0:
        raise ValueError("oracle_head_score rejected its arguments")
    return score


def bin_index(sprime: float, B: int) -> int:
    return int(lib().oracle_bin_index(float(sprime), int(B)))


def prob_map(score, q_lut=None):
    """sigmoid, bin index and posterior lookup (Appendix A.4).  Returns (prob, bin, q)."""
    score = np.ascontiguousarray(score, dtype=np.float64)
    N = score.shape[0]
    prob = np.empty(N, dtype=np.float64)
    q = np.empty(N, dtype=np.float64)
    bins = np.empty(N, dtype=np.int32)
    if q_lut is not None:
        q_lut = np.ascontiguousarray(q_lut, dtype=np.float32)
        B = q_lut.shape[0]
    else:
        B = 0
    lib().oracle_prob_map(_p(score), C.c_int(N), C.c_int(B), _p(q_lut), _p(prob), _p(bins), _p(q))
    return prob, bins, q


def calib_counts(sprime, y, B: int):
    sprime = np.ascontiguousarray(sprime, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.uint8)
    cpos = np.empty(B, dtype=np.int64)
    cneg = np.empty(B, dtype=np.int64)
    lib().oracle_calib_counts(_p(sprime), _p(y), C.c_int64(sprime.shape[0]), C.c_int(B), _p(cpos), _p(cneg))
    return cpos, cneg


def build_q_lut(cpos, cneg, alpha: float = 1.0):
    """Returns (q as float64 [B], q rounded once to float32 [B])."""
    cpos = np.ascontiguousarray(cpos, dtype=np.int64)
    cneg = np.ascontiguousarray(cneg, dtype=np.int64)
    B = cpos.shape[0]
    q64 = np.empty(B, dtype=np.float64)
    q32 = np.empty(B, dtype=np.float32)
    lib().oracle_build_q_lut(_p(cpos), _p(cneg), C.c_int(B), C.c_double(alpha), _p(q64), _p(q32))
    return q64, q32


def select(q, P: int, G: int, K: int, rho: float = 0.5, return_order: bool = False):
    """Exact-K per-group balancing selection (Section 4.1).  keep uint8 [P*G]."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    assert q.shape[0] == P * G
    keep = np.empty(P * G, dtype=np.uint8)
    order = np.empty(P * max(G - K, 0), dtype=np.int32) if return_order else None
    rc = lib().oracle_select(_p(q), C.c_int(P), C.c_int(G), C.c_int(K), C.c_double(rho), _p(keep), _p(order))
    if rc != 0:
        raise ValueError("oracle_select rejected its arguments")
    return (keep, order.reshape(P, max(G - K, 0))) if return_order else keep


def survivor_scan(keep, lengths):
    """Returns (survivor_idx int32 [S], cu_seqlens int64 [S+1], S, T)."""
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    N = keep.shape[0]
    idx = np.empty(N, dtype=np.int32)
    cu = np.empty(N + 1, dtype=np.int64)
    num = np.empty(2, dtype=np.int64)
    lib().oracle_survivor_scan(_p(keep), _p(lengths), C.c_int(N), _p(idx), _p(cu), _p(num))
    S, T = int(num[0]), int(num[1])
    return idx[:S].copy(), cu[:S + 1].copy(), S, T


def gather(survivor_idx, cu_seqlens, src_tok_off, src_tokens=None, src_rows=None):
    """Packed survivors: returns (dst_tokens, dst_rows as uint8 [T,row_bytes] or None, tok_seq)."""
    survivor_idx = np.ascontiguousarray(survivor_idx, dtype=np.int32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int64)
    off = np.ascontiguousarray(src_tok_off, dtype=np.int64)
    S = survivor_idx.shape[0]
    T = int(cu[S])
    dst_tokens = None
    if src_tokens is not None:
        src_tokens = np.ascontiguousarray(src_tokens, dtype=np.int32)
        dst_tokens = np.empty(T, dtype=np.int32)
    dst_rows = None
    row_bytes = 0
    if src_rows is not None:
        src_rows = np.ascontiguousarray(src_rows)
        src_rows = src_rows.view(np.uint8).reshape(src_rows.shape[0], -1)
        row_bytes = src_rows.shape[1]
        dst_rows = np.empty((T, row_bytes), dtype=np.uint8)
    tok_seq = np.empty(T, dtype=np.int32)
    lib().oracle_gather(_p(survivor_idx), _p(cu), C.c_int64(S), _p(off), _p(src_tokens), _p(src_rows),
                        C.c_int64(row_bytes), _p(dst_tokens), _p(dst_rows), _p(tok_seq))
    return dst_tokens, dst_rows, tok_seq


def advantages(rewards, keep, G: int, eps: float = 1e-6, ddof: int = 0):
    """Group-relative advantage on the survivors (Section 3), float64 [S] in survivor order."""
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    N = keep.shape[0]
    adv = np.zeros(int(keep.astype(np.int64).sum()), dtype=np.float64)
    lib().oracle_advantages(_p(rewards), _p(keep), C.c_int(N), C.c_int(G), C.c_double(eps), C.c_int(ddof),
                            _p(adv))
    return adv


def token_logprob(hidden, W, targets, rows=None, inv_temp: float = 1.0):
    """fp64 two-pass log-softmax gather (Section 3).  Returns (logp, lse) for `rows` (all rows if None)."""
    hidden = np.ascontiguousarray(hidden)
    code = _dtype_code(hidden)
    (W,) = _same_dtype(code, W)
    targets = np.ascontiguousarray(targets, dtype=np.int32)
    V, d = W.shape
    assert hidden.shape[1] == d
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        n = rows.shape[0]
    else:
        n = hidden.shape[0]
    logp = np.empty(n, dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    rc = lib().oracle_token_logprob(_p(hidden), _p(W), C.c_int(code), _p(targets), _p(rows), C.c_int64(n),
                                    C.c_int(d), C.c_int(V), C.c_double(inv_temp), _p(logp), _p(lse))
    if rc != 0:
        raise MemoryError("oracle_token_logprob could not allocate its scratch")
    return logp, lse


class ScoreBuffers:
    """Positive / negative sliding buffers of normalised scores (Appendix A.4), FIFO of `cap` entries each."""

    def __init__(self, cap: int):
        self.cap = int(cap)
        self.pos = np.zeros(cap, dtype=np.float64)
        self.neg = np.zeros(cap, dtype=np.float64)
        self.state = np.zeros(4, dtype=np.int64)      # head_pos, n_pos, head_neg, n_neg

    def push(self, sprime, y):
        sprime = np.ascontiguousarray(sprime, dtype=np.float64)
        y = np.ascontiguousarray(y, dtype=np.uint8)
        st = self.state
        P64 = C.POINTER(C.c_int64)
        base = st.ctypes.data
        ptr = lambda i: C.cast(base + 8 * i, P64)
        lib().oracle_buffer_push(_p(self.pos), ptr(0), ptr(1), _p(self.neg), ptr(2), ptr(3), C.c_int64(self.cap),
                                 _p(sprime), _p(y), C.c_int64(sprime.shape[0]))

    def contents(self):
        """(positive scores oldest..newest, negative scores oldest..newest)"""
        hp, n_p, hn, n_n = (int(v) for v in self.state)
        pos = np.array([self.pos[(hp + i) % self.cap] for i in range(n_p)])
        neg = np.array([self.neg[(hn + i) % self.cap] for i in range(n_n)])
        return pos, neg

    def counts(self, B: int):
        pos, neg = self.contents()
        s = np.concatenate([pos, neg])
        y = np.concatenate([np.ones(len(pos), np.uint8), np.zeros(len(neg), np.uint8)])
        return calib_counts(s, y, B)


def solve_delta(cpos, cneg, q_lut, kappa=0.5, lam=0.5, rho=0.5, p_min=0.05, p_max=0.95, iters=64) -> float:
    cpos = np.ascontiguousarray(cpos, dtype=np.int64)
    cneg = np.ascontiguousarray(cneg, dtype=np.int64)
    q_lut = np.ascontiguousarray(q_lut, dtype=np.float32)
    f = lib().oracle_solve_delta
    f.restype = C.c_double
    return float(f(_p(cpos), _p(cneg), _p(q_lut), C.c_int(q_lut.shape[0]), C.c_double(kappa), C.c_double(lam),
                   C.c_double(rho), C.c_double(p_min), C.c_double(p_max), C.c_int(iters)))


def select_stochastic(q, u, delta, eligible=None, kappa=0.5, lam=0.5, rho=0.5, p_min=0.05, p_max=0.95):
    """Returns (keep uint8 [N], p float64 [N])."""
    q = np.ascontiguousarray(q, dtype=np.float32)
    u = np.ascontiguousarray(u, dtype=np.float32)
    N = q.shape[0]
    if eligible is not None:
        eligible = np.ascontiguousarray(eligible, dtype=np.uint8)
    keep = np.empty(N, dtype=np.uint8)
    p = np.empty(N, dtype=np.float64)
    lib().oracle_select_stochastic(_p(q), _p(u), _p(eligible), C.c_int64(N), C.c_double(kappa), C.c_double(delta),
                                   C.c_double(lam), C.c_double(rho), C.c_double(p_min), C.c_double(p_max),
                                   _p(keep), _p(p))
    return keep, p
