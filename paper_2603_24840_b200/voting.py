"""ctypes binding of the test-time rank-weighted vote (marshalling only)."""
import ctypes as C

from . import binding as B


def arrol_rank_vote(ctx: B.Context, score, answer, P: int, G: int, weight, winner, winner_weight, stream=None):
    lib = B.load_library()
    lib.arrol_rank_vote.restype = C.c_int
    lib.arrol_rank_vote.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_void_p]
    B._check(lib.arrol_rank_vote(ctx.handle, B._ptr(score), B._ptr(answer), int(P), int(G), B._ptr(weight),
                                 B._ptr(winner), B._ptr(winner_weight), B._stream(stream)), "arrol_rank_vote")
