"""Pins for the CPU oracle: every check compares it with something that does not
come from the oracle itself -- a library softmax, exact rational arithmetic over
a dense weight matrix, enumeration against the exactness proposition of
Sec. 2.2, a hand-worked example, and a separately written token-level
speculative-sampling verifier.  A plausible slip in the oracle (dropped 1/N(t),
swapped ratio, wrong residual sign, draft instead of target inside the group,
wrong uniform) fails at least one of them.
"""
from fractions import Fraction

import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from paper_2511_13732_b200 import workloads as W


def _logits_from_probs(p):
    """float32 logits whose softmax is (up to float32 rounding of the logs) the given pmf."""
    return np.log(np.asarray(p, dtype=np.float64)).astype(np.float32)


def _dense_w(groups):
    """Dense equal-split weight matrix w[k, t] = 1{t in G_k}/N(t) as Fractions."""
    Wm = [[Fraction(0)] * groups.V for _ in range(groups.M)]
    for g in range(groups.M):
        for k in range(groups.group_ptr[g], groups.group_ptr[g + 1]):
            t = int(groups.group_tok[k])
            Wm[g][t] = Fraction(1, int(groups.tok_degree[t]))
    return Wm


# ---------------------------------------------------------------- softmax ----
@pytest.mark.parametrize("T", [1.0, 0.8, 2.5])
def test_softmax_matches_library_routine(oracle, T):
    rng = np.random.default_rng(1)
    x = (3.0 * rng.standard_normal((5, 97))).astype(np.float32)
    want = scipy_softmax(x.astype(np.float64) / np.float64(np.float32(T)), axis=1)
    np.testing.assert_allclose(oracle.softmax(x, T), want, rtol=1e-13, atol=0)


def test_softmax_bf16_bits_are_widened_exactly(oracle):
    rng = np.random.default_rng(2)
    bits = W.f32_to_bf16_bits((4.0 * rng.standard_normal((3, 64))).astype(np.float32))
    want = scipy_softmax(W.bf16_bits_to_f32(bits).astype(np.float64), axis=1)
    np.testing.assert_allclose(oracle.softmax(bits, 1.0), want, rtol=1e-13)


def test_softmax_fp16_values_are_widened_exactly(oracle):
    rng = np.random.default_rng(21)
    x = (4.0 * rng.standard_normal((3, 80))).astype(np.float16)
    x[0, :4] = np.array([6.0e-8, -6.0e-5, 65504.0, -np.inf], np.float16)  # subnormal, small normal, largest, mask
    x[0, 2] = np.float16(11.0)
    want = scipy_softmax(x.astype(np.float64), axis=1)
    np.testing.assert_allclose(oracle.softmax(x, 1.0), want, rtol=1e-13)
    # every finite binary16 pattern widens to the value numpy assigns to it (checked through a two-token softmax)
    bits = np.arange(0, 0x7C00, 37, dtype=np.uint16)
    vals = bits.view(np.float16)
    pair = np.stack([vals / np.float16(1.0), np.zeros_like(vals)], axis=1).astype(np.float16)
    got = oracle.softmax(pair[pair[:, 0] < 30], 1.0)
    v64 = pair[pair[:, 0] < 30][:, 0].astype(np.float64)
    np.testing.assert_allclose(got[:, 0], 1.0 / (1.0 + np.exp(-v64)), rtol=1e-13)


def test_softmax_handles_masked_tokens(oracle):
    x = np.array([[0.0, -np.inf, 1.0, -np.inf]], np.float32)
    p = oracle.softmax(x, 1.0)
    assert p[0, 1] == 0 and p[0, 3] == 0
    np.testing.assert_allclose(p[0, [0, 2]], [1 / (1 + np.e), np.e / (1 + np.e)], rtol=1e-14)


# ------------------------------------------------------- coarse-graining ----
def test_group_probs_exact_rationals():
    """Equal-split coarse-graining against exact rational arithmetic with a dense weight matrix."""
    import oracle

    groups = W.groups_from_lists(6, [[0, 1, 2], [2, 3], [1, 2, 4, 5], [5], []])
    p = [Fraction(1, 3), Fraction(1, 4), Fraction(1, 6), Fraction(1, 8), Fraction(1, 16), Fraction(1, 16)]
    assert sum(p) == 1
    Wm = _dense_w(groups)
    want = [sum(Wm[g][t] * p[t] for t in range(6)) for g in range(groups.M)]
    assert sum(want) == 1  # weights sum to one per token (Sec. 2.2)
    got = oracle.group_probs(_logits_from_probs([float(v) for v in p])[None, :], groups.group_ptr, groups.group_tok,
                             groups.tok_degree)
    np.testing.assert_allclose(got[0], [float(v) for v in want], rtol=0, atol=2e-7)
    assert got[0, 4] == 0.0  # an empty group has no mass


def test_group_probs_special_cases(oracle):
    rng = np.random.default_rng(3)
    x = (2.0 * rng.standard_normal((4, 50))).astype(np.float32)
    p = scipy_softmax(x.astype(np.float64), axis=1)
    single = W.groups_from_lists(50, [[t] for t in range(50)])
    np.testing.assert_allclose(oracle.group_probs(x, single.group_ptr, single.group_tok, single.tok_degree), p,
                               rtol=1e-13)
    one = W.groups_from_lists(50, [list(range(50))])
    np.testing.assert_allclose(oracle.group_probs(x, one.group_ptr, one.group_tok, one.tok_degree), 1.0, rtol=1e-13)
    # two identical groups split every token's mass in half
    dup = W.groups_from_lists(50, [list(range(50)), list(range(50))])
    np.testing.assert_allclose(oracle.group_probs(x, dup.group_ptr, dup.group_tok, dup.tok_degree), 0.5, rtol=1e-13)


@pytest.mark.parametrize("name", ["C1", "C2", "C4"])
def test_group_probs_sum_to_one_and_match_dense_matrix(oracle, name):
    cfg = W.scaled(W.CONFIGS[name], V=256, M=64, emb_dim=16) if name != "C4" else W.scaled(W.CONFIGS[name], V=512, M=96)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=2)
    rows = bt.draft_logits.reshape(-1, cfg.V)
    got = oracle.group_probs(rows, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=1e-12)
    dense = np.zeros((groups.M, cfg.V))
    for g in range(groups.M):
        toks = groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
        dense[g, toks] = 1.0 / groups.tok_degree[toks]
    val = W.bf16_bits_to_f32(rows) if cfg.dtype == "bf16" else rows
    p = scipy_softmax(val.astype(np.float64) / np.float64(np.float32(cfg.temperature)), axis=1)
    np.testing.assert_allclose(got, p @ dense.T, rtol=1e-11, atol=1e-300)
    # coarse-graining can only raise the overlap: sum_g min(P,Q) >= sum_t min(p,q)
    tgt = bt.target_logits[:, :cfg.K].reshape(-1, cfg.V)
    P = oracle.group_probs(tgt, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    tv = W.bf16_bits_to_f32(tgt) if cfg.dtype == "bf16" else tgt
    pt = scipy_softmax(tv.astype(np.float64) / np.float64(np.float32(cfg.temperature)), axis=1)
    assert np.all(np.minimum(P, got).sum(axis=1) >= np.minimum(pt, p).sum(axis=1) - 1e-12)


def test_general_weights_reduce_to_equal_split(oracle):
    groups = W.groups_from_lists(6, [[0, 1, 2], [2, 3], [1, 2, 4, 5], [5]])
    x = np.random.default_rng(4).standard_normal((3, 6)).astype(np.float32)
    w = 1.0 / groups.tok_degree[groups.group_tok]
    a = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree)
    b = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, weights=w)
    np.testing.assert_allclose(a, b, rtol=1e-14)


# ------------------------------------------------ hand-worked example ----
# V = 4, groups G0 = {0,1}, G1 = {1,2}, G2 = {3}; N = (1,2,1,1).
# target p = (1/2, 1/4, 1/8, 1/8), draft q = (1/8, 1/8, 1/4, 1/2).
# P = (1/2 + 1/8, 1/8 + 1/8, 1/8) = (5/8, 1/4, 1/8);  Q = (1/8 + 1/16, 1/16 + 1/4, 1/2) = (3/16, 5/16, 1/2).
# Draft token x = 1 lies in G0 and G1: label G0 if u_label < 1/2 (P0 >= Q0: always accepted), else G1 with
# ratio (1/4)/(5/16) = 0.8.  Residual (P-Q)_+ = (7/16, 0, 0): the resampled group is G0 whatever the uniform;
# inside G0 the weights are p0/1 = 1/2 and p1/2 = 1/8, so token 0 iff u_token < 0.8.
# Bonus (all accepted): group from P = (5/8, 1/4, 1/8) by inverse CDF, token inside it by the same rule.
HAND = W.groups_from_lists(4, [[0, 1], [1, 2], [3]])
HAND_P = [0.5, 0.25, 0.125, 0.125]
HAND_Q = [0.125, 0.125, 0.25, 0.5]


def _hand_case(oracle, u_label, u_accept, u_group, u_token, bonus_p=None):
    tgt = np.stack([_logits_from_probs(HAND_P), _logits_from_probs(bonus_p or HAND_P)])[None]
    drf = _logits_from_probs(HAND_Q)[None, None]
    u = np.array([[[u_label, u_accept], [u_group, u_token]]], np.float32)
    return oracle.verify(tgt, drf, np.array([[1]], np.int32), HAND.group_ptr, HAND.group_tok, HAND.tok_degree, u)


def test_hand_worked_example(oracle):
    r = _hand_case(oracle, 0.25, 0.99, 0.7, 0.5)  # label G0: accepted although u_accept is large
    assert r.accept_len[0] == 1 and r.groups[0, 0] == 0 and r.tokens[0, 0] == 1
    r = _hand_case(oracle, 0.75, 0.79, 0.7, 0.6)  # label G1, 0.79 < 0.8: accepted; bonus group from P: 0.7 -> G1
    assert r.accept_len[0] == 1 and r.groups[0, 0] == 1 and r.tokens[0, 0] == 1
    assert r.groups[0, 1] == 1  # 5/8 <= 0.7 < 7/8
    # inside G1 = {1,2}: weights p1/2 = 1/8 and p2/1 = 1/8, so u_token 0.6 picks token 2
    assert r.tokens[0, 1] == 2
    r = _hand_case(oracle, 0.75, 0.81, 0.999, 0.79)  # label G1, 0.81 >= 0.8: rejected; residual is all on G0
    assert r.accept_len[0] == 0 and r.groups[0, 0] == 0 and r.tokens[0, 0] == 0
    assert r.tokens[0, 1] == -1 and r.groups[0, 1] == -1
    np.testing.assert_allclose(r.margins[0, 0, 1], 0.01, atol=1e-6)
    r = _hand_case(oracle, 0.75, 0.81, 0.0, 0.81)  # same, token draw beyond 0.8 -> token 1
    assert r.accept_len[0] == 0 and r.tokens[0, 0] == 1
    r = _hand_case(oracle, 0.25, 0.0, 0.9, 0.3)  # bonus: 0.9 >= 7/8 -> G2 = {3}
    assert r.accept_len[0] == 1 and r.groups[0, 1] == 2 and r.tokens[0, 1] == 3


# ------------------------------------- exactness proposition by enumeration ----
def _tiny_problem(seed):
    rng = np.random.default_rng(seed)
    groups = W.groups_from_lists(6, [[0, 1, 2], [2, 3], [1, 2, 4, 5], [5, 0]])
    tl = (1.5 * rng.standard_normal((2, 6))).astype(np.float32)  # position 0 and the bonus row
    dl = (1.5 * rng.standard_normal((1, 6))).astype(np.float32)
    p = scipy_softmax(tl.astype(np.float64), axis=1)
    q = scipy_softmax(dl.astype(np.float64), axis=1)[0]
    Wm = np.array([[float(v) for v in row] for row in _dense_w(groups)])
    return groups, tl, dl, p, q, Wm


def _run_grid(oracle, groups, tl, dl, xs, u_label, u_accept, u_group, u_token):
    """Run the oracle on the full factorial of the given draft tokens and uniform grids (K = 1)."""
    mesh = np.meshgrid(xs, u_label, u_accept, u_group, u_token, indexing="ij")
    flat = [m.reshape(-1) for m in mesh]
    B = flat[0].size
    u = np.empty((B, 2, 2), np.float32)
    u[:, 0, 0], u[:, 0, 1], u[:, 1, 0], u[:, 1, 1] = flat[1], flat[2], flat[3], flat[4]
    res = oracle.verify(np.broadcast_to(tl, (B, 2, 6)).copy(), np.broadcast_to(dl, (B, 1, 6)).copy(),
                        flat[0].astype(np.int32)[:, None], groups.group_ptr, groups.group_tok, groups.tok_degree, u,
                        threads=0)
    return flat[0].astype(int), res, mesh[0].shape


def _midpoints(n):
    return (np.arange(n) + 0.5) / n


@pytest.mark.parametrize("seed", [11, 12])
def test_label_coupling_and_acceptance_probability(oracle, seed):
    """Pr(label = k) equals the draft coarse mass, and Pr(accept, label = k) = min(P_k, Q_k) (proof of the proposition)."""
    groups, tl, dl, p, q, Wm = _tiny_problem(seed)
    P, Q = Wm @ p[0], Wm @ q
    NL, NA = 12, 2000  # 12 is a multiple of every degree here, so the label grid is exact
    xs, res, _ = _run_grid(oracle, groups, tl, dl, np.arange(6), _midpoints(NL), _midpoints(NA), [0.5], [0.5])
    wgt = q[xs] / (NL * NA)
    label = np.where(res.accept_len == 1, res.groups[:, 0], -2)
    # the label of a rejected position is overwritten by the resampled group, so recover it from a second run
    # with an accept uniform of 0 (every label with positive ratio is then accepted)
    xs2, res2, _ = _run_grid(oracle, groups, tl, dl, np.arange(6), _midpoints(NL), [0.0], [0.5], [0.5])
    assert np.all(res2.accept_len == 1)
    lab_hist = np.bincount(res2.groups[:, 0], weights=q[xs2] / NL, minlength=groups.M)
    np.testing.assert_allclose(lab_hist, Q, rtol=1e-6)
    for x, g in zip(xs2, res2.groups[:, 0]):
        assert x in groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
    acc_hist = np.bincount(label[label >= 0], weights=wgt[label >= 0], minlength=groups.M)
    np.testing.assert_allclose(acc_hist, np.minimum(P, Q), atol=1.0 / NA)
    # overall acceptance probability is 1 - TV(P, Q)
    np.testing.assert_allclose(acc_hist.sum(), 1.0 - 0.5 * np.abs(P - Q).sum(), atol=4.0 / NA)


@pytest.mark.parametrize("seed", [11, 13])
def test_residual_group_law_and_emitted_group_is_target_coarse(oracle, seed):
    """Reject branch draws from (P-Q)_+/TV; accepted plus resampled groups together follow P exactly (proposition)."""
    groups, tl, dl, p, q, Wm = _tiny_problem(seed)
    P, Q = Wm @ p[0], Wm @ q
    resid = np.maximum(P - Q, 0)
    # a label whose group has P < Q, forced to reject with an accept uniform just below 1
    k_rej = int(np.argmax(Q - P))
    x = int(groups.group_tok[groups.group_ptr[k_rej]])
    S = [g for g in range(groups.M) if x in groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]]
    u_lab = (S.index(k_rej) + 0.5) / len(S)
    NG = 4000
    _, res, _ = _run_grid(oracle, groups, tl, dl, [x], [u_lab], [1.0 - 2.0 ** -24], _midpoints(NG), [0.5])
    if P[k_rej] > 0 and (1.0 - 2.0 ** -24) < P[k_rej] / Q[k_rej]:
        pytest.skip("ratio too close to one to force a rejection")
    assert np.all(res.accept_len == 0)
    hist = np.bincount(res.groups[:, 0], minlength=groups.M) / NG
    np.testing.assert_allclose(hist, resid / resid.sum(), atol=1.5 / NG)
    assert np.all(res.flags == 0)
    # joint enumeration: emitted group at position 0 is distributed as the target coarse distribution P
    NL, NA, NG2 = 12, 160, 160
    xs, res, _ = _run_grid(oracle, groups, tl, dl, np.arange(6), _midpoints(NL), _midpoints(NA), _midpoints(NG2), [0.5])
    emitted = np.bincount(res.groups[:, 0], weights=q[xs] / (NL * NA * NG2), minlength=groups.M)
    np.testing.assert_allclose(emitted, P, atol=2.0 / NA + 2.0 / NG2)
    np.testing.assert_allclose(emitted.sum(), 1.0, rtol=1e-9)


@pytest.mark.parametrize("seed", [11, 14])
def test_within_group_and_bonus_token_law(oracle, seed):
    """Token inside the resampled group follows the target conditional; the bonus token follows the target p."""
    groups, tl, dl, p, q, Wm = _tiny_problem(seed)
    NG, NT = 300, 300
    # accept uniform 0: every position is accepted, the terminal draw is the bonus from target row 1
    xs, res, _ = _run_grid(oracle, groups, tl, dl, [int(np.argmax(q))], [0.5], [0.0], _midpoints(NG), _midpoints(NT))
    assert np.all(res.accept_len == 1)
    tok_hist = np.bincount(res.tokens[:, 1], minlength=6) / (NG * NT)
    np.testing.assert_allclose(tok_hist, p[1], atol=2.0 / NG + 2.0 / NT)
    grp_hist = np.bincount(res.groups[:, 1], minlength=groups.M) / (NG * NT)
    np.testing.assert_allclose(grp_hist, Wm @ p[1], atol=1.5 / NG)
    # conditional on the group: p(t) w / P[g]
    for g in range(groups.M):
        sel = res.groups[:, 1] == g
        if sel.sum() == 0:
            continue
        cond = np.bincount(res.tokens[sel, 1], minlength=6) / sel.sum()
        want = Wm[g] * p[1] / (Wm[g] @ p[1])
        np.testing.assert_allclose(cond, want, atol=3.0 / NT + 3.0 / NG)
        assert np.all(cond[Wm[g] == 0] == 0)  # the emitted token always lies in the emitted group


# -------------------- disjoint groups reduce to token-level speculative sampling ----
def _textbook_sd(p, q, x, u):
    """Standard speculative sampling for one sequence, written independently of the oracle.
    p [K+1, n], q [K, n] pmfs; x [K] drafted items; u [K+1, 2] uniforms (column 1 of rows < K = accept draw,
    u[K, 0] = terminal draw).  Returns (accept length, emitted item at the terminal position)."""
    K = q.shape[0]
    for i in range(K):
        if q[i, x[i]] > 0 and not (p[i, x[i]] >= q[i, x[i]]) and not (u[i, 1] < p[i, x[i]] / q[i, x[i]]):
            r = np.maximum(p[i] - q[i], 0.0)
            c = np.cumsum(r)
            return i, int(np.searchsorted(c, np.float64(u[K, 0]) * c[-1], side="right"))
    c = np.cumsum(p[K])
    return K, int(np.searchsorted(c, np.float64(u[K, 0]) * c[-1], side="right"))


def test_singleton_groups_equal_textbook_speculative_sampling(oracle):
    rng = np.random.default_rng(21)
    B, K, V = 200, 5, 40
    tl = (2.0 * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    dl = (tl[:, :K] + rng.standard_normal((B, K, V))).astype(np.float32)
    q = scipy_softmax(dl.astype(np.float64), axis=2)
    p = scipy_softmax(tl.astype(np.float64), axis=2)
    x = np.array([[rng.choice(V, p=q[b, i]) for i in range(K)] for b in range(B)], np.int32)
    u = rng.random((B, K + 1, 2)).astype(np.float32)
    g = W.groups_from_lists(V, [[t] for t in range(V)])
    res = oracle.verify(tl, dl, x, g.group_ptr, g.group_tok, g.tok_degree, u)
    lens = []
    for b in range(B):
        n, z = _textbook_sd(p[b], q[b], x[b], u[b])
        lens.append(n)
        assert res.accept_len[b] == n
        assert res.tokens[b, n] == z and res.groups[b, n] == z
        assert np.array_equal(res.tokens[b, :n], x[b, :n]) and np.all(res.tokens[b, n + 1:] == -1)
    assert 0 < np.mean(lens) < K  # both branches are exercised
    assert K in lens and 0 in lens


def test_partition_groups_equal_textbook_sampling_on_lumped_distributions(oracle):
    rng = np.random.default_rng(22)
    B, K, V, M = 200, 4, 60, 12
    assign = rng.integers(0, M, size=V)
    assign[:M] = np.arange(M)
    g = W.groups_from_lists(V, [list(np.nonzero(assign == k)[0]) for k in range(M)])
    tl = (2.0 * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    dl = (tl[:, :K] + 1.5 * rng.standard_normal((B, K, V))).astype(np.float32)
    p = scipy_softmax(tl.astype(np.float64), axis=2)
    q = scipy_softmax(dl.astype(np.float64), axis=2)
    lump = np.zeros((V, M))
    lump[np.arange(V), assign] = 1.0
    x = np.array([[rng.choice(V, p=q[b, i]) for i in range(K)] for b in range(B)], np.int32)
    u = rng.random((B, K + 1, 2)).astype(np.float32)
    res = oracle.verify(tl, dl, x, g.group_ptr, g.group_tok, g.tok_degree, u)
    for b in range(B):
        n, gz = _textbook_sd(p[b] @ lump, q[b] @ lump, assign[x[b]], u[b])
        assert res.accept_len[b] == n and res.groups[b, n] == gz
        assert np.array_equal(res.groups[b, :n], assign[x[b, :n]])
        assert assign[res.tokens[b, n]] == gz


# -------------------------------------------------- structure on workloads ----
@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_emission_structure_on_workloads(oracle, name):
    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=min(cfg.B, 8))
    res = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                        groups.tok_degree, bt.uniforms, bt.temperature, threads=0)
    for b in range(bt.draft_tokens.shape[0]):
        n = res.accept_len[b]
        assert 0 <= n <= cfg.K
        assert np.array_equal(res.tokens[b, :n], bt.draft_tokens[b, :n])  # accepted draft tokens are kept
        assert np.all(res.tokens[b, n + 1:] == -1) and np.all(res.groups[b, n + 1:] == -1)
        for i in range(n + 1):  # every emitted token lies in its emitted group
            g = res.groups[b, i]
            assert res.tokens[b, i] in groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
    # same inputs, any thread count: identical outputs
    res1 = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                         groups.tok_degree, bt.uniforms, bt.temperature, threads=1)
    assert np.array_equal(res.tokens, res1.tokens) and np.array_equal(res.accept_len, res1.accept_len)


def test_oracle_rejects_invalid_membership(oracle):
    g = W.groups_from_lists(4, [[0, 1], [1, 2]])  # token 3 is in no group: N(3) = 0
    x = np.zeros((1, 2, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.verify(x, x[:, :1], np.zeros((1, 1), np.int32), g.group_ptr, g.group_tok, g.tok_degree,
                      np.zeros((1, 2, 2), np.float32))
