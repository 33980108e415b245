"""GPU parity: every step of the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Integer / byte / index results are compared bit for bit; floating results within the stated tolerances
(probabilities 1e-3, advantages 1e-5, token log-probs 2e-3, all absolute)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_24840_b200 import binding as B
from paper_2603_24840_b200 import synth
from paper_2603_24840_b200.pipeline import PruneRebatch, host_inputs

pytestmark = pytest.mark.gpu

PROB_TOL = 1e-3
ADV_TOL = 1e-5
LOGP_TOL = 2e-3


@pytest.fixture(scope="module")
def ctx():
    c = B.Context(0)
    yield c
    assert B.arrol_poll_status(c, raise_on_error=False) == 0    # no test leaves a device status behind
    c.close()


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)) if isinstance(a, np.ndarray) else a
    return t.cuda() if dtype is None else t.cuda().to(dtype)


# ------------------------------------------------------------------------------------------------------------
# a1 + a2: quality head and probability map
# ------------------------------------------------------------------------------------------------------------
def _score_case(ctx, N, d, h, dtype, use_lut, use_index, seed, bias=True):
    g = np.random.default_rng(seed)
    rows = N * 3 if use_index else N
    x = torch.from_numpy(g.normal(size=(rows, d)).astype(np.float32)).to(dtype)
    mk = lambda *s: torch.from_numpy(g.normal(0, 0.05, size=s).astype(np.float32)).to(dtype)
    if h == 0:
        head = {"W1": mk(d), "b1": mk(1) if bias else None, "w2": None, "b2": None}
    else:
        head = {"W1": mk(h, d), "b1": mk(h) if bias else None, "w2": mk(h) * 4, "b2": mk(1) if bias else None}
    ridx = g.permutation(rows)[:N].astype(np.int64) if use_index else None
    lut = None
    if use_lut:
        s, y = synth.calib_history(synth.WORKLOADS["tiny"])
        cpos, cneg = oracle.calib_counts(s, y, 128)
        _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    s_ref = oracle.head_score(oa(x), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]),
                              row_index=ridx, h=h)
    p_ref, b_ref, q_ref = oracle.prob_map(s_ref, lut)

    dhead = {k: (None if v is None else v.cuda()) for k, v in head.items()}
    dhead["h"] = h
    score = torch.full((N,), 7.0, device="cuda")
    prob = torch.full((N,), 7.0, device="cuda")
    q = torch.full((N,), 7.0, device="cuda")
    bins = torch.full((N,), -5, dtype=torch.int32, device="cuda")
    B.arrol_score_partial(ctx, x.cuda(), dhead, N, score, prob, q, bin=bins,
                          row_index=None if ridx is None else dev(ridx), q_lut=None if lut is None else dev(lut))
    torch.cuda.synchronize()
    score, prob, q, bins = score.cpu().numpy(), prob.cpu().numpy(), q.cpu().numpy(), bins.cpu().numpy()
    assert np.abs(score - s_ref).max() <= PROB_TOL
    assert np.abs(prob - p_ref).max() <= PROB_TOL
    if lut is None:
        assert np.array_equal(q, prob)
    else:
        Bn = 128
        # the bin is decided on the kernel's own fp32 s' (128 s' is exact in fp32 and fp64): same decision rule
        assert np.array_equal(bins, np.array([oracle.bin_index(float(v), Bn) for v in prob]))
        assert np.array_equal(q, lut[bins])                                  # bit-equal table lookup
        near_edge = np.abs(Bn * p_ref - np.rint(Bn * p_ref)) <= Bn * PROB_TOL
        assert np.all((bins == b_ref) | (near_edge & (np.abs(bins - b_ref) <= 1)))


@pytest.mark.parametrize("N,d,dtype,use_lut,use_index", [
    (32, 256, torch.float32, False, False),
    (32, 256, torch.float32, True, True),
    (513, 2048, torch.bfloat16, True, True),
    (77, 2560, torch.bfloat16, True, False),
    (5, 8, torch.bfloat16, False, False),
    (130, 4096 + 64, torch.bfloat16, True, True),
])
def test_linear_head(ctx, N, d, dtype, use_lut, use_index):
    _score_case(ctx, N, d, 0, dtype, use_lut, use_index, seed=N + d)
    _score_case(ctx, N, d, 0, dtype, use_lut, use_index, seed=N + d + 1, bias=False)


@pytest.mark.parametrize("N,d,h,dtype", [
    (48, 192, 24, torch.bfloat16),
    (300, 2048, 256, torch.bfloat16),
    (70, 264, 132, torch.float32),
    (129, 512, 512, torch.bfloat16),
    (1000, 1024, 128, torch.bfloat16),      # several 128-row tiles and K ranges on the tensor-core path
    (257, 200, 68, torch.bfloat16),         # d and h off the 64-wide tile edges
    (2048, 2048, 256, torch.bfloat16),      # the Qwen-3-1.7B-shaped head
    (40, 64, 64, torch.bfloat16),           # one K step: three of the four MMA issuers have nothing to do
    (33, 128, 16, torch.bfloat16),          # two K steps
    (17, 8, 4, torch.bfloat16),             # a K step of 8 columns, 4 hidden units
    (4096, 4096, 512, torch.bfloat16),      # the DAPO-shaped head over all prompts (256 blocks: more than one wave)
])
def test_mlp_head(ctx, N, d, h, dtype):
    _score_case(ctx, N, d, h, dtype, True, True, seed=N + h)
    _score_case(ctx, N, d, h, dtype, False, False, seed=N + h + 1, bias=False)


def test_mlp_head_larger_than_the_packing_buffer_takes_the_simt_path(ctx):
    """N * d * 2 bytes beyond the context's 64 MB row-packing buffer: the call falls back to the fp32 SIMT kernels
    (same results); without a row index the rows are tiled in place and no packing is needed."""
    _score_case(ctx, 8448, 4096, 64, torch.bfloat16, False, True, seed=3)     # 69 MB of scored rows, indexed
    _score_case(ctx, 8448, 4096, 64, torch.bfloat16, True, False, seed=4)     # same size, rows in place


def test_mlp_head_strided_rows_without_index(ctx):
    """Evenly strided rows (a column slice of a wider buffer) go to the tensor-core path without packing."""
    g = np.random.default_rng(5)
    N, d, h = 200, 256, 64
    wide = torch.from_numpy(g.normal(size=(N, 2 * d)).astype(np.float32)).to(torch.bfloat16)
    x = wide[:, :d]
    mk = lambda *s: torch.from_numpy(g.normal(0, 0.05, size=s).astype(np.float32)).to(torch.bfloat16)
    head = {"W1": mk(h, d), "b1": mk(h), "w2": mk(h) * 4, "b2": mk(1)}
    oa = synth.as_oracle_array
    s_ref = oracle.head_score(oa(x.contiguous()), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]), h=h)
    dhead = {k: v.cuda() for k, v in head.items()}
    dhead["h"] = h
    out = [torch.full((N,), 7.0, device="cuda") for _ in range(3)]
    B.arrol_score_partial(ctx, wide.cuda()[:, :d], dhead, N, out[0], out[1], out[2])
    torch.cuda.synchronize()
    assert np.abs(out[0].cpu().numpy() - s_ref).max() <= PROB_TOL


def test_score_argument_errors(ctx):
    x = torch.zeros(4, 16, device="cuda")
    out = torch.zeros(4, device="cuda")
    head = {"W1": torch.zeros(16, device="cuda"), "b1": None, "w2": None, "b2": None, "h": 0}
    B.arrol_score_partial(ctx, x, head, 0, out, out, out)                    # N = 0: no-op
    with pytest.raises(B.ArrolError) as e:
        B.arrol_score_partial(ctx, x[:, :12], dict(head, W1=torch.zeros(12, device="cuda")), 4, out, out, out)
    assert e.value.code == -2                                               # d % 8 != 0
    with pytest.raises(B.ArrolError) as e:
        B.arrol_score_partial(ctx, x, dict(head, W1=None), 4, out, out, out)
    assert e.value.code == -1


# ------------------------------------------------------------------------------------------------------------
# a3: selection, fed the oracle's q: bit-exact
# ------------------------------------------------------------------------------------------------------------
def _select_both(ctx, q, P, G, K, rho):
    ref = oracle.select(q, P, G, K, rho)
    keep = torch.full((P * G,), 9, dtype=torch.uint8, device="cuda")
    B.arrol_select(ctx, dev(q), P, G, K, rho, keep)
    torch.cuda.synchronize()
    assert np.array_equal(keep.cpu().numpy(), ref)


def test_select_every_group_size(ctx):
    g = np.random.default_rng(0)
    for G in range(1, 33):
        P = 37
        for qs in (g.random(P * G), g.integers(0, 17, size=P * G) / 16, g.beta(0.5, 0.5, size=P * G)):
            q = qs.astype(np.float32)
            for K in sorted({1, max(1, G // 2), max(1, G - 1), G}):
                _select_both(ctx, q, P, G, K, 0.5)
        _select_both(ctx, g.random(P * G).astype(np.float32), P, G, max(1, G // 2), 0.3)


def test_select_on_table_valued_q_and_constants(ctx):
    # q = q_lut[bin] takes at most 128 values: many exact ties
    w = synth.WORKLOADS["qwen3-1.7b"]
    s, y = synth.calib_history(w)
    cpos, cneg = oracle.calib_counts(s, y, 128)
    _, lut = oracle.build_q_lut(cpos, cneg, 1.0)
    g = np.random.default_rng(1)
    q = lut[g.integers(0, 128, size=w.N)]
    _select_both(ctx, q, w.P, w.G, w.K, 0.5)
    for val in (0.0, 0.5, 1.0):
        _select_both(ctx, np.full(16 * 5, val, np.float32), 5, 16, 8, 0.5)
    tiny = np.array([1e-30, 3e-9, 1.0, 0.5, 2e-38, 0.25, 0.75, 1e-12] * 3, np.float32)   # sums that round
    _select_both(ctx, tiny, 3, 8, 4, 0.5)


def test_select_argument_errors(ctx):
    q = torch.zeros(64, device="cuda")
    keep = torch.zeros(64, dtype=torch.uint8, device="cuda")
    for (P, G, K, mode), code in {(1, 64, 8, 0): -2, (4, 16, 0, 0): -1, (4, 16, 17, 0): -1, (4, 16, 8, 1): -2}.items():
        with pytest.raises(B.ArrolError) as e:
            B.arrol_select(ctx, q, P, G, K, 0.5, keep, mode=mode)
        assert e.value.code == code
    B.arrol_select(ctx, q, 0, 16, 8, 0.5, keep)                             # P = 0: no-op


# ------------------------------------------------------------------------------------------------------------
# a4-a6: scan, gather, advantages
# ------------------------------------------------------------------------------------------------------------
def _compact_case(ctx, N, G, row_bytes, seed, keep_prob=0.5, lo=0, hi=40, padded=False, ddof=0, with_tokens=True,
                  cap_slack=3):
    g = np.random.default_rng(seed)
    ell = g.integers(lo, hi + 1, size=N).astype(np.int32)
    keep = (g.random(N) < keep_prob).astype(np.uint8)
    rewards = (g.random(N) < 0.4).astype(np.float32)
    if padded:
        off = (np.arange(N, dtype=np.int64) * (hi + 3))
        T_src = N * (hi + 3)
    else:
        off_full = synth.src_offsets(ell)
        off, T_src = off_full[:-1], int(off_full[-1])
    T_src = max(T_src, 1)
    tokens = g.integers(0, 1 << 30, size=T_src).astype(np.int32)
    rows = g.integers(0, 256, size=(T_src, row_bytes)).astype(np.uint8) if row_bytes else None

    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    dt_ref, dr_ref, seq_ref = oracle.gather(idx, cu, off, tokens if with_tokens else None, rows)
    adv_ref = oracle.advantages(rewards, keep, G, eps=1e-6, ddof=ddof)

    cap = T + cap_slack
    d_idx = torch.full((N,), -1, dtype=torch.int32, device="cuda")
    d_cu = torch.full((N + 1,), -1, dtype=torch.int64, device="cuda")
    d_adv = torch.full((N,), 99.0, device="cuda")
    d_num = torch.full((2,), -1, dtype=torch.int64, device="cuda")
    d_tok = torch.full((cap,), -7, dtype=torch.int32, device="cuda") if with_tokens else None
    d_rows = torch.full((cap, row_bytes), 255, dtype=torch.uint8, device="cuda") if row_bytes else None
    d_tadv = torch.full((cap,), 99.0, device="cuda")
    d_tseq = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    B.arrol_compact(ctx, dev(keep), dev(ell), dev(off), N, G, dev(rewards), cap, d_cu, d_idx, d_adv, d_num,
                    src_tokens=dev(tokens) if with_tokens else None, dst_tokens=d_tok,
                    src_rows=dev(rows) if row_bytes else None, dst_rows=d_rows, row_bytes=row_bytes,
                    tok_adv=d_tadv, tok_seq=d_tseq, ddof=ddof)
    torch.cuda.synchronize()
    assert d_num.cpu().tolist() == [S, T]
    assert np.array_equal(d_idx.cpu().numpy()[:S], idx)
    assert np.array_equal(d_cu.cpu().numpy()[:S + 1], cu)
    adv = d_adv.cpu().numpy()[:S]
    assert np.abs(adv - adv_ref).max(initial=0.0) <= ADV_TOL
    if with_tokens:
        assert np.array_equal(d_tok.cpu().numpy()[:T], dt_ref)
        assert np.all(d_tok.cpu().numpy()[T:] == -7)                         # nothing written past T
    assert np.array_equal(d_tseq.cpu().numpy()[:T], seq_ref)
    assert np.array_equal(d_tadv.cpu().numpy()[:T], adv[seq_ref]) if T else True
    if row_bytes:
        assert np.array_equal(d_rows.cpu().numpy()[:T], dr_ref)
        assert np.all(d_rows.cpu().numpy()[T:] == 255)
    return S, T


@pytest.mark.parametrize("N,G,row_bytes", [(32, 8, 0), (32, 8, 1024), (2048, 16, 64), (4096, 16, 0),
                                           (5000, 8, 16), (96, 32, 4096), (48, 16, 8192 + 16),
                                           (24, 8, 32768), (24, 8, 32768 + 64)])   # largest bulk-copy row; load/store kernel
def test_compact_matches_oracle(ctx, N, G, row_bytes):
    _compact_case(ctx, N, G, row_bytes, seed=N + row_bytes)
    _compact_case(ctx, N, G, row_bytes, seed=N + row_bytes + 1, padded=True, ddof=1)


def test_compact_edge_cases(ctx):
    assert _compact_case(ctx, 64, 8, 32, seed=1, keep_prob=0.0) == (0, 0)            # nobody survives
    _compact_case(ctx, 64, 8, 32, seed=2, keep_prob=1.1)                              # everybody survives: identity
    _compact_case(ctx, 64, 8, 32, seed=3, lo=0, hi=2)                                 # many zero-length rollouts
    _compact_case(ctx, 64, 8, 48, seed=4, cap_slack=0)                                # capacity exactly T
    _compact_case(ctx, 16, 16, 0, seed=5, with_tokens=False)                          # scan outputs only
    _compact_case(ctx, 1030, 1, 16, seed=6, lo=1, hi=3)                               # groups of one: adv = 0
    _compact_case(ctx, 3000, 8, 32, seed=7, lo=300, hi=700)                           # ~0.75M tokens, many tiles


def test_compact_degenerate_groups_and_capacity_overflow(ctx):
    G, N = 8, 24
    rewards = np.array([0] * G + [1] * G + [1, 0] * (G // 2), np.float32)
    keep = np.ones(N, np.uint8)
    ell = np.full(N, 5, np.int32)
    off = synth.src_offsets(ell)[:-1]
    tokens = np.arange(N * 5, dtype=np.int32)
    outs = dict(cu=torch.zeros(N + 1, dtype=torch.int64, device="cuda"),
                idx=torch.zeros(N, dtype=torch.int32, device="cuda"), adv=torch.ones(N, device="cuda"),
                num=torch.zeros(2, dtype=torch.int64, device="cuda"))
    dst = torch.full((N * 5,), -1, dtype=torch.int32, device="cuda")
    B.arrol_compact(ctx, dev(keep), dev(ell), dev(off), N, G, dev(rewards), N * 5, outs["cu"], outs["idx"],
                    outs["adv"], outs["num"], src_tokens=dev(tokens), dst_tokens=dst)
    torch.cuda.synchronize()
    adv = outs["adv"].cpu().numpy()
    assert np.all(adv[:2 * G] == 0.0) and np.all(adv[2 * G:] != 0.0)          # all-0 / all-1 groups: exactly zero
    assert np.array_equal(dst.cpu().numpy(), tokens)
    # destination one row too small: scan outputs written, nothing gathered, status recorded, no fault
    dst.fill_(-1)
    B.arrol_compact(ctx, dev(keep), dev(ell), dev(off), N, G, dev(rewards), N * 5 - 1, outs["cu"], outs["idx"],
                    outs["adv"], outs["num"], src_tokens=dev(tokens), dst_tokens=dst[:N * 5 - 1])
    bits = B.arrol_poll_status(ctx, raise_on_error=False)
    assert bits == B.DEV_CAPACITY
    assert outs["num"].cpu().tolist() == [N, N * 5] and np.all(dst.cpu().numpy() == -1)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0                # cleared by the poll
    with pytest.raises(B.ArrolError) as e:                                    # N not a multiple of G
        B.arrol_compact(ctx, dev(keep), dev(ell), dev(off), N, 7, dev(rewards), 10, outs["cu"], outs["idx"],
                        outs["adv"], outs["num"])
    assert e.value.code == -1


# ------------------------------------------------------------------------------------------------------------
# a7: fused lm_head log-prob
# ------------------------------------------------------------------------------------------------------------
def _logprob_case(ctx, T, d, V, seed, scale=1.0, wstd=0.05, T_live=None, inv_temp=1.0, sample=None, edge_targets=True):
    g = np.random.default_rng(seed)
    H = torch.from_numpy((g.normal(size=(T, d)) * scale).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(g.normal(0, wstd, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    y = g.integers(0, V, size=T).astype(np.int32)
    if edge_targets:
        edges = [0, V - 1, min(127, V - 1), min(128, V - 1), min(255, V - 1), min(256, V - 1), (V - 1) // 256 * 256, -1]
        y[:min(T, len(edges))] = edges[:min(T, len(edges))]
        if T > 20:
            y[T - 1] = V - 1
            y[T // 2] = -3
    n_live = T if T_live is None else min(T_live, T)
    rows = np.arange(n_live) if sample is None else np.unique(np.concatenate(
        [np.arange(min(8, n_live)), [n_live - 1], g.integers(0, n_live, size=sample)]))
    rows = rows.astype(np.int64)
    lp_ref, lse_ref = oracle.token_logprob(synth.as_oracle_array(H), synth.as_oracle_array(W), y, rows=rows,
                                           inv_temp=inv_temp)
    logp = torch.full((T,), 55.0, device="cuda")
    lse = torch.full((T,), 55.0, device="cuda")
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    d_T = None if T_live is None else torch.tensor([T_live], dtype=torch.int64, device="cuda")
    B.arrol_token_logprob(ctx, H.cuda(), W.cuda(), dev(y), T, d, V, logp, ws, lse=lse, d_T=d_T,
                          inv_temperature=inv_temp)
    torch.cuda.synchronize()
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    logp, lse = logp.cpu().numpy(), lse.cpu().numpy()
    assert np.abs(logp[rows] - lp_ref).max(initial=0.0) <= LOGP_TOL
    assert np.abs(lse[rows] - lse_ref).max(initial=0.0) <= LOGP_TOL
    assert np.all(logp[rows][y[rows] < 0] == 0.0)
    if T_live is not None:
        assert np.all(logp[n_live:] == 55.0) and np.all(lse[n_live:] == 55.0)   # rows past T are not written
    return logp


@pytest.mark.parametrize("T,d,V", [
    (1, 64, 256), (128, 64, 256), (129, 64, 512), (300, 192, 1000), (257, 200, 37), (2900, 256, 4096),
    (1000, 512, 5000), (333, 2048, 1500), (64, 4096, 777),
])
def test_token_logprob_matches_oracle(ctx, T, d, V):
    _logprob_case(ctx, T, d, V, seed=T + d + V)


def test_token_logprob_dominant_logits_temperature_and_device_T(ctx):
    _logprob_case(ctx, 200, 256, 3000, seed=1, scale=30.0)                   # one logit dominates: lse ~ max
    _logprob_case(ctx, 200, 256, 3000, seed=2, inv_temp=0.6)
    _logprob_case(ctx, 500, 128, 1024, seed=3, T_live=301)                   # T read from the device, ragged tile
    _logprob_case(ctx, 500, 128, 1024, seed=4, T_live=0)
    _logprob_case(ctx, 400, 128, 1024, seed=5, T_live=4000)                  # *d_T larger than T_max is clamped


def test_token_logprob_unsplit_and_split_paths_agree_with_oracle(ctx):
    # many token tiles, small d: one vocabulary split per tile (direct write path)
    _logprob_case(ctx, 19200, 64, 512, seed=6, sample=200)
    # few token tiles, many chunks: the vocabulary is split across thread blocks and merged
    _logprob_case(ctx, 130, 128, 20000, seed=7)


def test_token_logprob_uniform_and_invariances(ctx):
    T, d, V = 256, 128, 1111
    g = np.random.default_rng(8)
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    y = torch.from_numpy(g.integers(0, V, size=T).astype(np.int32)).cuda()
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    logp = torch.empty(T, device="cuda")
    B.arrol_token_logprob(ctx, torch.zeros(T, d, dtype=torch.bfloat16, device="cuda"), W, y, T, d, V, logp, ws)
    torch.cuda.synchronize()
    assert np.abs(logp.cpu().numpy() + np.log(V)).max() <= 1e-5              # zero hidden state: -log V
    # permuting the vocabulary rows (and the targets) leaves log-probs unchanged up to summation order
    H = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    perm = torch.from_numpy(g.permutation(V)).cuda()
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(V, device="cuda")
    lp1 = torch.empty(T, device="cuda")
    lp2 = torch.empty(T, device="cuda")
    B.arrol_token_logprob(ctx, H, W, y, T, d, V, lp1, ws)
    B.arrol_token_logprob(ctx, H, W[perm].contiguous(), inv[y.long()].int(), T, d, V, lp2, ws)
    torch.cuda.synchronize()
    assert (lp1 - lp2).abs().max().item() <= 1e-4


def test_token_logprob_bad_target_and_argument_errors(ctx):
    T, d, V = 130, 64, 300
    H = torch.zeros(T, d, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(V, d, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, dtype=torch.int32, device="cuda")
    y[5] = V          # outside the vocabulary
    logp = torch.full((T,), 3.0, device="cuda")
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    B.arrol_token_logprob(ctx, H, W, y, T, d, V, logp, ws)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == B.DEV_BAD_TARGET
    assert logp[5].item() == 0.0 and abs(logp[4].item() + np.log(V)) < 1e-5
    with pytest.raises(B.ArrolError) as e:
        B.arrol_token_logprob(ctx, H, W, y, T, d, V, logp, None)
    assert e.value.code == -3
    with pytest.raises(B.ArrolError) as e:
        B.arrol_token_logprob(ctx, H, W, y, T, 60, V, logp, ws)
    assert e.value.code == -2
    with pytest.raises(B.ArrolError) as e:
        B.arrol_token_logprob(ctx, H, W, y, T, d, V, logp, ws, inv_temperature=0.0)
    assert e.value.code == -1
    B.arrol_token_logprob(ctx, H, W, y, 0, d, V, logp, ws)                    # T_max = 0: no-op


# ------------------------------------------------------------------------------------------------------------
# whole path on workload shapes
# ------------------------------------------------------------------------------------------------------------
def _pipeline_parity(name, n_logp_rows):
    w = synth.WORKLOADS[name]
    inp = host_inputs(w, with_hidden=True)
    pr = PruneRebatch(w, inputs=inp)
    pr.step()
    torch.cuda.synchronize()
    assert B.arrol_poll_status(pr.ctx, raise_on_error=False) == 0
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    head = inp["head"]
    ridx = inp["src_tok_off"][:-1] + (w.cutoff - 1)
    s_ref = oracle.head_score(oa(inp["hidden"]), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]),
                              row_index=ridx, h=w.h)
    hs, hy = inp["calib_history"]
    _, lut = oracle.build_q_lut(*oracle.calib_counts(hs, hy, w.B), 1.0)
    assert np.array_equal(lut, inp["q_lut"])
    p_ref, b_ref, _ = oracle.prob_map(s_ref, lut)
    assert np.abs(pr.prob.cpu().numpy() - p_ref).max() <= PROB_TOL
    # downstream steps are compared on the GPU's own q (what the pipeline consumed): selection is bit-exact
    q_gpu = pr.q.cpu().numpy()
    keep_ref = oracle.select(q_gpu, w.P, w.G, w.K, w.rho)
    assert np.array_equal(pr.keep.cpu().numpy(), keep_ref)
    idx, cu, S, T = oracle.survivor_scan(keep_ref, inp["lengths"])
    assert pr.counts() == (S, T) and S == w.S
    assert np.array_equal(pr.survivor_idx.cpu().numpy()[:S], idx)
    assert np.array_equal(pr.cu_seqlens.cpu().numpy()[:S + 1], cu)
    rows_src = inp["hidden"].to(torch.bfloat16)
    dt_ref, dr_ref, seq_ref = oracle.gather(idx, cu, inp["src_tok_off"][:-1], inp["src_tokens"], oa(rows_src))
    assert np.array_equal(pr.dst_tokens.cpu().numpy()[:T], dt_ref)
    assert np.array_equal(pr.dst_rows.view(torch.uint8).cpu().numpy()[:T], dr_ref)
    assert np.array_equal(pr.tok_seq.cpu().numpy()[:T], seq_ref)
    adv_ref = oracle.advantages(inp["rewards"], keep_ref, w.G)
    assert np.abs(pr.adv.cpu().numpy()[:S] - adv_ref).max() <= ADV_TOL
    # selected-token log-probs on the packed survivors
    g = np.random.default_rng(0)
    rows = np.arange(T) if n_logp_rows is None else np.unique(np.concatenate(
        [[0, T - 1], cu[:-1][::16], cu[1:][::16] - 1, g.integers(0, T, size=n_logp_rows)]))
    packed = dr_ref.view(np.uint16).reshape(T, w.d)
    lp_ref, lse_ref = oracle.token_logprob(packed, oa(inp["W_vocab"]), dt_ref, rows=rows)
    assert np.abs(pr.logp.cpu().numpy()[rows] - lp_ref).max() <= LOGP_TOL
    assert np.abs(pr.lse.cpu().numpy()[rows] - lse_ref).max() <= LOGP_TOL


def test_whole_path_tiny():
    _pipeline_parity("tiny", None)


def test_whole_path_mini():
    _pipeline_parity("mini", None)


@pytest.mark.parametrize("T,d,V,splits", [(300, 64, 300, 0), (1000, 192, 3000, 0), (128 * 148 * 2 + 77, 64, 520, 0),
                                          (128 * 148 + 5, 64, 1100, 3), (700, 128, 2000, 2)])
def test_pairs_of_blocks_and_single_blocks_give_the_same_logprobs(T, d, V, splits):
    """The log-prob kernel as clusters of two blocks on 256-row tiles (the default) against one block per 128-row tile:
    the same products in the same order, so the same bits; both within 2e-3 of the oracle.  Covers a single partial
    wave, several waves (the blocks wait for one another per wave), an odd number of token tiles, forced splits."""
    ctx = B.Context(0)
    if splits:
        B.arrol_test_hook(ctx, B.HOOK_LOGPROB_SPLITS, splits)
    g = np.random.default_rng(T + V)
    H = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16)
    y = g.integers(0, V, size=T).astype(np.int32)
    out = []
    for pair in (1, 0):
        B.arrol_test_hook(ctx, B.HOOK_LOGPROB_PAIR, pair)
        ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
        lp = torch.full((T,), 7.0, device="cuda")
        lse = torch.full((T,), 7.0, device="cuda")
        B.arrol_token_logprob(ctx, H.cuda(), W.cuda(), dev(y), T, d, V, lp, ws, lse=lse)
        torch.cuda.synchronize()
        out.append((lp, lse))
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    assert torch.equal(out[0][0], out[1][0]) and torch.equal(out[0][1], out[1][1])
    rows = np.unique(np.concatenate([[0, T - 1, min(T - 1, 127), min(T - 1, 128), min(T - 1, 255), min(T - 1, 256)],
                                     g.integers(0, T, size=40)])).astype(np.int64)
    lp_ref, lse_ref = oracle.token_logprob(synth.as_oracle_array(H), synth.as_oracle_array(W), y, rows=rows)
    assert np.abs(out[0][0].cpu().numpy()[rows] - lp_ref).max() <= LOGP_TOL
    assert np.abs(out[0][1].cpu().numpy()[rows] - lse_ref).max() <= LOGP_TOL
    ctx.close()


def test_logprob_call_replayed_from_a_cuda_graph():
    """arrol_token_logprob allocates nothing and never synchronises: a launch of several waves (the wave counter is
    cleared by a memset node, a cluster launch) can be captured once and replayed."""
    ctx = B.Context(0)
    g = np.random.default_rng(11)
    T, d, V = 128 * 148 * 2 + 300, 64, 777
    H = torch.from_numpy(g.normal(size=(T, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    y = dev(g.integers(0, V, size=T).astype(np.int32))
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T, d, V), dtype=torch.uint8, device="cuda")
    ref = torch.full((T,), 7.0, device="cuda")
    B.arrol_token_logprob(ctx, H, W, y, T, d, V, ref, ws)
    torch.cuda.synchronize()
    lp = torch.full((T,), 7.0, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        B.arrol_token_logprob(ctx, H, W, y, T, d, V, lp, ws, stream=side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        B.arrol_token_logprob(ctx, H, W, y, T, d, V, lp, ws, stream=side)
    for _ in range(2):
        lp.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(lp, ref)
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    del graph
    ctx.close()


@pytest.mark.parametrize("T_live", [0, 1, 129, 148 * 128 + 5, 2 * 148 * 128 + 300])
def test_logprob_device_side_count_below_a_capacity_of_several_waves(T_live):
    """The launch is sized for T_max (more than two waves of token tiles, so the blocks are held in step), the live count
    comes from device memory: fewer waves than the host planned, blocks without a work item, nothing written past T."""
    ctx = B.Context(0)
    g = np.random.default_rng(12)
    T_max, d, V = 2 * 148 * 128 + 300, 64, 600
    H = torch.from_numpy(g.normal(size=(T_max, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    W = torch.from_numpy(g.normal(0, 0.05, size=(V, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    y = dev(g.integers(0, V, size=T_max).astype(np.int32))
    ws = torch.empty(B.arrol_token_logprob_workspace(ctx, T_max, d, V), dtype=torch.uint8, device="cuda")
    full = torch.empty(T_max, device="cuda")
    B.arrol_token_logprob(ctx, H, W, y, T_max, d, V, full, ws)
    d_T = torch.tensor([T_live], dtype=torch.int64, device="cuda")
    lp = torch.full((T_max,), 7.0, device="cuda")
    lse = torch.full((T_max,), 7.0, device="cuda")
    for _ in range(2):
        B.arrol_token_logprob(ctx, H, W, y, T_max, d, V, lp, ws, lse=lse, d_T=d_T)
    torch.cuda.synchronize()
    assert torch.equal(lp[:T_live], full[:T_live])          # same tiles, same splits: the same bits
    assert torch.all(lp[T_live:] == 7.0) and torch.all(lse[T_live:] == 7.0)
    rows = np.unique(np.concatenate([[0, max(T_live - 1, 0)], g.integers(0, max(T_live, 1), size=6)]))[: max(min(T_live, 8), 0)]
    if T_live:
        ref, _ = oracle.token_logprob(synth.as_oracle_array(H[torch.from_numpy(rows).cuda()].cpu()),
                                      synth.as_oracle_array(W.cpu()), y.cpu().numpy()[rows])
        assert np.abs(lp.cpu().numpy()[rows] - ref).max() <= 2e-3
    assert B.arrol_poll_status(ctx, raise_on_error=False) == 0
    ctx.close()
