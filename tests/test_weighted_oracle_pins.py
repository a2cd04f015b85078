"""Pins for the oracle's general-weights branches (the weight equation of Sec. 2.2: w_{k,t} >= 0, zero off the
group, summing to one over the groups of each token) with UNEQUAL weights, and for the constant acceptance bias of
the lossy comparison system of Sec. 3.2.

Nothing here comes from the oracle: expected values are exact rationals over a dense weight matrix typed in by
hand, the identities the paper states (label law Pr(K = k) = sum_t q(t) w_{k,t}; Pr(accept, k) = min(P_k, Q_k);
emitted group ~ P; token inside the group ~ p(t) w_{K,t} / P_K), and labels written out by hand.
"""
from fractions import Fraction as F

import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

# V = 6 tokens, M = 4 groups.  Dense weights w[k][t], columns sum to one; zero = token not in the group.
#            t=0       t=1       t=2       t=3   t=4   t=5
DENSE = [[F(3, 4), F(1, 5), F(1, 2), 0, 0, 0],          # G0 = {0, 1, 2}
         [0, 0, F(1, 3), F(1), 0, 0],                   # G1 = {2, 3}
         [0, F(4, 5), F(1, 6), 0, F(1), F(2, 3)],       # G2 = {1, 2, 4, 5}
         [F(1, 4), 0, 0, 0, 0, F(1, 3)]]                # G3 = {0, 5}
LISTS = [[0, 1, 2], [2, 3], [1, 2, 4, 5], [0, 5]]
GROUPS = W.groups_from_lists(6, LISTS)
# the same weights in the order of the stored (group, token) pairs
PAIR_W = np.array([float(DENSE[g][t]) for g, toks in enumerate(LISTS) for t in toks])
WM = np.array([[float(v) for v in row] for row in DENSE])
# target (position 0 and bonus row) and draft pmfs as exact rationals
P0 = [F(1, 3), F(1, 4), F(1, 6), F(1, 8), F(1, 16), F(1, 16)]
P1 = [F(1, 16), F(1, 16), F(1, 8), F(1, 4), F(1, 6), F(1, 3)]
Q0 = [F(1, 12), F(1, 12), F(1, 3), F(1, 4), F(1, 8), F(1, 8)]


def _logits(p):
    return np.log(np.array([float(v) for v in p], np.float64)).astype(np.float32)


def _coarse(p):
    return [sum(DENSE[g][t] * p[t] for t in range(6)) for g in range(4)]


def _midpoints(n):
    return (np.arange(n) + 0.5) / n


def _run_grid(oracle, xs, u_label, u_accept, u_group, u_token, bias=0.0, weights=PAIR_W):
    mesh = np.meshgrid(xs, u_label, u_accept, u_group, u_token, indexing="ij")
    flat = [m.reshape(-1) for m in mesh]
    B = flat[0].size
    u = np.empty((B, 2, 2), np.float32)
    u[:, 0, 0], u[:, 0, 1], u[:, 1, 0], u[:, 1, 1] = flat[1], flat[2], flat[3], flat[4]
    tl = np.broadcast_to(np.stack([_logits(P0), _logits(P1)]), (B, 2, 6)).copy()
    dl = np.broadcast_to(_logits(Q0), (B, 1, 6)).copy()
    res = oracle.verify(tl, dl, flat[0].astype(np.int32)[:, None], GROUPS.group_ptr, GROUPS.group_tok,
                        GROUPS.tok_degree, u, weights=weights, accept_bias=bias, threads=0)
    return flat[0].astype(int), res


def test_the_hand_made_weights_are_a_valid_split():
    for t in range(6):
        assert sum(DENSE[g][t] for g in range(4)) == 1
        for g in range(4):
            assert (DENSE[g][t] != 0) == (t in LISTS[g])
    assert sum(_coarse(P0)) == 1 and sum(_coarse(Q0)) == 1  # no renormalisation needed (Sec. 2.2)


def test_weighted_group_probs_exact_rationals(oracle):
    want = [float(v) for v in _coarse(P0)]
    got = oracle.group_probs(_logits(P0)[None, :], GROUPS.group_ptr, GROUPS.group_tok, GROUPS.tok_degree, weights=PAIR_W)
    np.testing.assert_allclose(got[0], want, rtol=0, atol=2e-7)
    # and they differ from the equal split, so the weights really are used
    eq = oracle.group_probs(_logits(P0)[None, :], GROUPS.group_ptr, GROUPS.group_tok, GROUPS.tok_degree)
    assert np.abs(eq[0] - np.array(want)).max() > 0.02


def test_weighted_label_draw_hand_cases(oracle):
    """Token 2 lies in G0, G1, G2 with weights 1/2, 1/3, 1/6: label G0 below 1/2, G1 below 5/6, else G2.
    Token 5 lies in G2, G3 with weights 2/3, 1/3.  Token 0 in G0, G3 with 3/4, 1/4.  Accept uniform 0."""
    cases = [(2, 0.1, 0), (2, 0.49, 0), (2, 0.51, 1), (2, 0.83, 1), (2, 0.84, 2), (2, 0.99, 2),
             (5, 0.6, 2), (5, 0.7, 3), (0, 0.74, 0), (0, 0.76, 3), (3, 0.5, 1), (4, 0.999, 2)]
    for x, ul, want in cases:
        _, res = _run_grid(oracle, [x], [ul], [0.0], [0.5], [0.5])
        assert res.accept_len[0] == 1 and res.groups[0, 0] == want, (x, ul, want, res.groups[0])


def test_weighted_label_law_and_acceptance_law(oracle):
    """Pr(K = k) = sum_t q(t) w_{k,t} = Q_k (the coupling identity) and Pr(accept, K = k) = min(P_k, Q_k)."""
    P = np.array([float(v) for v in _coarse(P0)])
    Q = np.array([float(v) for v in _coarse(Q0)])
    q = np.array([float(v) for v in Q0])
    NL = 3000  # every label boundary (multiples of 1/2, 1/3, 1/4, 1/5, 1/6) is a grid edge: the label grid is exact
    xs, res = _run_grid(oracle, np.arange(6), _midpoints(NL), [0.0], [0.5], [0.5])
    assert np.all(res.accept_len == 1)
    lab = np.bincount(res.groups[:, 0], weights=q[xs] / NL, minlength=4)
    np.testing.assert_allclose(lab, Q, rtol=1e-6)
    NL2, NA = 60, 1500
    xs, res = _run_grid(oracle, np.arange(6), _midpoints(NL2), _midpoints(NA), [0.5], [0.5])
    acc = res.accept_len == 1
    hist = np.bincount(res.groups[acc, 0], weights=(q[xs] / (NL2 * NA))[acc], minlength=4)
    np.testing.assert_allclose(hist, np.minimum(P, Q), atol=1.0 / NA)
    np.testing.assert_allclose(hist.sum(), 1.0 - 0.5 * np.abs(P - Q).sum(), atol=4.0 / NA)


def test_weighted_emitted_group_is_target_coarse(oracle):
    """The proposition with unequal weights: accepted labels and resampled groups together follow P exactly."""
    P = np.array([float(v) for v in _coarse(P0)])
    Q = np.array([float(v) for v in _coarse(Q0)])
    q = np.array([float(v) for v in Q0])
    NL, NA, NG = 60, 120, 120
    xs, res = _run_grid(oracle, np.arange(6), _midpoints(NL), _midpoints(NA), _midpoints(NG), [0.5])
    emitted = np.bincount(res.groups[:, 0], weights=q[xs] / (NL * NA * NG), minlength=4)
    np.testing.assert_allclose(emitted, P, atol=2.0 / NA + 2.0 / NG)
    # the reject branch alone: normalised residual
    resid = np.maximum(P - Q, 0.0)
    rej = res.accept_len == 0
    hist = np.bincount(res.groups[rej, 0], weights=(q[xs])[rej], minlength=4)
    np.testing.assert_allclose(hist / hist.sum(), resid / resid.sum(), atol=3.0 / NG)
    assert np.all(hist[resid == 0] == 0)


def test_weighted_within_group_and_bonus_token_law(oracle):
    """Token inside group K follows p(t) w_{K,t} / P_K; drawn after K ~ P this gives back the target p."""
    p1 = np.array([float(v) for v in P1])
    NG, NT = 360, 360
    xs, res = _run_grid(oracle, [2], [0.1], [0.0], _midpoints(NG), _midpoints(NT))
    assert np.all(res.accept_len == 1)
    tok = np.bincount(res.tokens[:, 1], minlength=6) / (NG * NT)
    np.testing.assert_allclose(tok, p1, atol=2.0 / NG + 2.0 / NT)
    grp = np.bincount(res.groups[:, 1], minlength=4) / (NG * NT)
    np.testing.assert_allclose(grp, WM @ p1, atol=1.5 / NG)
    for g in range(4):
        sel = res.groups[:, 1] == g
        cond = np.bincount(res.tokens[sel, 1], minlength=6) / sel.sum()
        want = WM[g] * p1 / (WM[g] @ p1)
        np.testing.assert_allclose(cond, want, atol=3.0 / NT + 3.0 / NG)
        assert np.all(cond[WM[g] == 0] == 0)
    # hand case: bonus row P1, group G3 = {0, 5}: terms p(0) w = 1/16 * 1/4 = 1/64 and p(5) w = 1/3 * 1/3 = 1/9,
    # so token 0 iff u_token < (1/64) / (1/64 + 1/9) = 9/73 = 0.1233
    P1c = [float(v) for v in _coarse(P1)]
    u_g3 = float(P1c[0] + P1c[1] + P1c[2] + 0.5 * P1c[3])
    for ut, want in ((0.12, 0), (0.13, 5)):
        _, r = _run_grid(oracle, [2], [0.1], [0.0], [u_g3], [ut])
        assert r.groups[0, 1] == 3 and r.tokens[0, 1] == want


@pytest.mark.parametrize("bias", [0.3, 0.05])
def test_acceptance_bias_law(oracle, bias):
    """Constant bias on the acceptance probability (the comparison system of Sec. 3.2): accept iff
    u < min(1, P_k/Q_k) + bias, so Pr(accept, K = k) = min(Q_k, P_k + bias Q_k).  Equal split and weights."""
    q = np.array([float(v) for v in Q0])
    for weights, Wd in ((PAIR_W, WM), (None, None)):
        if weights is None:
            Wd = np.zeros((4, 6))
            for g, toks in enumerate(LISTS):
                for t in toks:
                    Wd[g, t] = 1.0 / GROUPS.tok_degree[t]
        P = Wd @ np.array([float(v) for v in P0])
        Q = Wd @ q
        NL, NA = 60, 2000
        xs, res = _run_grid(oracle, np.arange(6), _midpoints(NL), _midpoints(NA), [0.5], [0.5], bias=bias, weights=weights)
        acc = res.accept_len == 1
        hist = np.bincount(res.groups[acc, 0], weights=(q[xs] / (NL * NA))[acc], minlength=4)
        np.testing.assert_allclose(hist, np.minimum(Q, P + bias * Q), atol=1.0 / NA)
        # the bias changes nothing but the accept test: a rejected sequence still draws from (P - Q)_+
        rej = ~acc
        assert np.all(np.maximum(P - Q, 0.0)[res.groups[rej, 0]] > 0)
    # hand case: token 3 lies in G1 alone; equal split P_1 = 1/6/3 + 1/8 = 13/72, Q_1 = 1/3/3 + 1/4 = 13/36: ratio 1/2
    for ua, want in ((0.79, 1), (0.81, 0)):
        _, r = _run_grid(oracle, [3], [0.5], [ua], [0.5], [0.5], bias=0.3, weights=None)
        assert r.accept_len[0] == want
