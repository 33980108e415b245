"""numpy front-end of the oracle's test-time voting (test infrastructure only)."""
import ctypes as C

import numpy as np

from . import _p, lib


def rank_vote(score, answer, P: int, G: int):
    """Returns (weight float64 [P*G], winner int32 [P], winner_weight float64 [P])."""
    assert G <= 1024
    score = np.ascontiguousarray(score, dtype=np.float32)
    answer = np.ascontiguousarray(answer, dtype=np.int32)
    weight = np.empty(P * G, dtype=np.float64)
    winner = np.empty(P, dtype=np.int32)
    ww = np.empty(P, dtype=np.float64)
    lib().oracle_rank_vote(_p(score), _p(answer), C.c_int(P), C.c_int(G), _p(weight), _p(winner), _p(ww))
    return weight, winner, ww
