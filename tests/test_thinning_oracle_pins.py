"""Pins for the oracle's thinning sampler (the thinning paragraph of the paper's Sec. 2.2).

Nothing here re-types the sampler.  The checks are the facts the paper states about it, measured on the oracle's
output over many seeded random uniforms (tolerances are five standard deviations of the estimate):
  * after a rejection the kept group follows the normalised residual (P - Q)_+ and, together with the accepted
    labels, the emitted group follows the target's coarse distribution exactly (the proposition);
  * the expected number of trials after a rejection is 1 / TV(P, Q);
  * the token inside the kept group follows the target-conditional p(t) w / P[g];
  * after an all-accepted sequence one candidate is drawn and the bonus token follows the target p;
  * singleton groups give token-level residual sampling (p - q)_+;
  * when every supplied trial is turned down the result is the enumerated draw (pinned on its own elsewhere);
  * uniforms of trials that are never reached do not matter;
  * the order in which the candidate draw walks the tokens is an INPUT (a permutation; None = ascending token id).
    The paper fixes the law y ~ target, which no order can change: the law pins run under the identity and under
    seeded random permutations; that the given order is really the one walked is checked against literal expected
    tokens on hand-made targets.
"""
import numpy as np
import pytest
from scipy.special import softmax as scipy_softmax

from paper_2511_13732_b200 import workloads as W
from test_oracle_pins import _dense_w, _tiny_problem

FLAG_EXHAUSTED = 8


def _uniforms(rng, shape):
    return (rng.integers(0, 1 << 24, size=shape) * 2.0 ** -24).astype(np.float32)


# candidate orders the law pins run under: ascending token id, and two seeded random permutations
ORDERS = [None, 101, 102]


def _order(which, V):
    return None if which is None else np.random.default_rng(which).permutation(V).astype(np.int32)


def _run(oracle, groups, tl, dl, x, u, tu, order=None):
    B = x.shape[0]
    V = tl.shape[-1]
    return oracle.verify(np.broadcast_to(tl, (B,) + tl.shape[-2:]).copy(), np.broadcast_to(dl, (B,) + dl.shape[-2:]).copy(),
                         x.astype(np.int32).reshape(B, -1), groups.group_ptr, groups.group_tok, groups.tok_degree, u,
                         thin_uniforms=tu, threads=0, cand_order=_order(order, V))


def _five_sigma(prob, n):
    return 5.0 * np.sqrt(np.maximum(prob * (1.0 - prob), 1e-4) / n) + 1e-9


@pytest.mark.parametrize("seed,order", [(11, None), (13, None), (11, 101), (13, 102)])
def test_thinning_group_law_trials_and_token_law(oracle, seed, order):
    groups, tl, dl, p, q, Wm = _tiny_problem(seed)
    P, Q = Wm @ p[0], Wm @ q
    resid = np.maximum(P - Q, 0.0)
    TV = resid.sum()
    rng = np.random.default_rng(1000 + seed)
    N, NTR = 300_000, 64
    x = rng.choice(6, size=N, p=q)
    u = _uniforms(rng, (N, 2, 2))
    tu = _uniforms(rng, (N, NTR, 3))
    res = _run(oracle, groups, tl, dl, x, u, tu, order)
    rej = res.accept_len == 0
    nrej = int(rej.sum())
    assert nrej > 0.5 * TV * N  # Pr(reject) = TV(P, Q)
    np.testing.assert_allclose(nrej / N, TV, atol=_five_sigma(TV, N))
    # the proposition: accepted labels and resampled groups together follow the target's coarse distribution
    emitted = np.bincount(res.groups[:, 0], minlength=groups.M) / N
    np.testing.assert_allclose(emitted, P, atol=_five_sigma(P, N).max())
    # the reject branch alone follows the normalised residual
    hist = np.bincount(res.groups[rej, 0], minlength=groups.M) / nrej
    np.testing.assert_allclose(hist, resid / TV, atol=_five_sigma(resid / TV, nrej).max())
    assert np.all(hist[resid == 0] == 0)
    # expected number of trials is 1 / TV (geometric with success probability TV)
    exhausted = (res.flags & FLAG_EXHAUSTED) != 0
    assert exhausted.sum() <= max(3, 10 * N * (1 - TV) ** NTR)
    tr = res.trials[rej & ~exhausted].astype(np.float64)
    np.testing.assert_allclose(tr.mean(), 1.0 / TV, atol=5.0 * np.sqrt(1.0 - TV) / TV / np.sqrt(tr.size) + 1e-3)
    assert np.all(res.trials[~rej] == 1)  # position accepted: the terminal draw is the bonus, one candidate
    # token inside the kept group: target-conditional p(t) w / P[g]
    for g in range(groups.M):
        sel = rej & (res.groups[:, 0] == g)
        if sel.sum() < 2000:
            continue
        cond = np.bincount(res.tokens[sel, 0], minlength=6) / sel.sum()
        want = Wm[g] * p[0] / (Wm[g] @ p[0])
        np.testing.assert_allclose(cond, want, atol=_five_sigma(want, sel.sum()).max())
        assert np.all(cond[Wm[g] == 0] == 0)


@pytest.mark.parametrize("seed,order", [(11, None), (14, None), (14, 101)])
def test_thinning_bonus_is_one_candidate_from_the_target(oracle, seed, order):
    groups, tl, dl, p, q, Wm = _tiny_problem(seed)
    rng = np.random.default_rng(2000 + seed)
    N = 200_000
    x = np.full(N, int(np.argmax(q)))
    u = _uniforms(rng, (N, 2, 2))
    u[:, 0, 1] = 0.0  # accept uniform 0: the drafted position is always accepted
    tu = _uniforms(rng, (N, 3, 3))
    res = _run(oracle, groups, tl, dl, x, u, tu, order)
    assert np.all(res.accept_len == 1) and np.all(res.trials == 1) and np.all(res.flags == 0)
    grp = np.bincount(res.groups[:, 1], minlength=groups.M) / N
    np.testing.assert_allclose(grp, Wm @ p[1], atol=_five_sigma(Wm @ p[1], N).max())
    tok = np.bincount(res.tokens[:, 1], minlength=6) / N
    np.testing.assert_allclose(tok, p[1], atol=_five_sigma(p[1], N).max())
    # the bonus candidate never looks at its third uniform
    tu2 = tu.copy()
    tu2[:, 0, 2] = 1.0 - 2.0 ** -24
    res2 = _run(oracle, groups, tl, dl, x, u, tu2, order)
    assert np.array_equal(res2.tokens, res.tokens) and np.array_equal(res2.groups, res.groups)


@pytest.mark.parametrize("order", ORDERS[:2])
def test_thinning_with_singleton_groups_is_token_level_residual_sampling(oracle, order):
    rng = np.random.default_rng(31)
    V = 7
    tl = (1.5 * rng.standard_normal((2, V))).astype(np.float32)
    dl = (1.5 * rng.standard_normal((1, V))).astype(np.float32)
    p = scipy_softmax(tl.astype(np.float64), axis=1)[0]
    q = scipy_softmax(dl.astype(np.float64), axis=1)[0]
    g = W.groups_from_lists(V, [[t] for t in range(V)])
    N = 200_000
    x = rng.choice(V, size=N, p=q)
    res = _run(oracle, g, tl, dl, x, _uniforms(rng, (N, 2, 2)), _uniforms(rng, (N, 64, 3)), order)
    rej = res.accept_len == 0
    resid = np.maximum(p - q, 0.0)
    hist = np.bincount(res.tokens[rej, 0], minlength=V) / rej.sum()
    np.testing.assert_allclose(hist, resid / resid.sum(), atol=_five_sigma(resid / resid.sum(), rej.sum()).max())
    assert np.array_equal(res.tokens[rej, 0], res.groups[rej, 0])
    emitted = np.bincount(res.tokens[:, 0], minlength=V) / N  # speculative sampling is exact at token level
    np.testing.assert_allclose(emitted, p, atol=_five_sigma(p, N).max())


def test_thinning_exhaustion_falls_back_to_the_enumerated_draw(oracle):
    groups, tl, dl, p, q, Wm = _tiny_problem(12)
    rng = np.random.default_rng(41)
    N = 4000
    x = rng.choice(6, size=N, p=q)
    u = _uniforms(rng, (N, 2, 2))
    tu = _uniforms(rng, (N, 2, 3))
    tu[:, :, 2] = 1.0 - 2.0 ** -24  # no candidate can be kept (every a(k) is below 1 here)
    res = _run(oracle, groups, tl, dl, x, u, tu)
    ref = oracle.verify(np.broadcast_to(tl, (N, 2, 6)).copy(), np.broadcast_to(dl, (N, 1, 6)).copy(),
                        x.astype(np.int32)[:, None], groups.group_ptr, groups.group_tok, groups.tok_degree, u, threads=0)
    rej = ref.accept_len == 0
    assert rej.sum() > 100
    assert np.array_equal(res.accept_len, ref.accept_len)
    assert np.array_equal(res.tokens[rej], ref.tokens[rej]) and np.array_equal(res.groups[rej], ref.groups[rej])
    assert np.all((res.flags[rej] & FLAG_EXHAUSTED) != 0) and np.all(res.trials[rej] == 2)
    assert np.all((res.flags[~rej] & FLAG_EXHAUSTED) == 0) and np.all(res.trials[~rej] == 1)


def test_thinning_never_reads_trials_it_does_not_reach(oracle):
    groups, tl, dl, p, q, Wm = _tiny_problem(13)
    rng = np.random.default_rng(51)
    N, NTR = 3000, 16
    x = rng.choice(6, size=N, p=q)
    u = _uniforms(rng, (N, 2, 2))
    tu = _uniforms(rng, (N, NTR, 3))
    res = _run(oracle, groups, tl, dl, x, u, tu)
    tu2 = tu.copy()
    for b in range(N):
        tu2[b, res.trials[b]:] = _uniforms(rng, (NTR - res.trials[b], 3))
    res2 = _run(oracle, groups, tl, dl, x, u, tu2)
    assert np.array_equal(res2.tokens, res.tokens) and np.array_equal(res2.groups, res.groups)
    assert np.array_equal(res2.trials, res.trials)
    assert res.trials.max() > 2  # several candidates were needed somewhere
    # and the trials it does reach matter: swapping the first candidate's token uniform changes some results
    tu3 = tu.copy()
    tu3[:, 0, 0] = _uniforms(rng, (N,))
    res3 = _run(oracle, groups, tl, dl, x, u, tu3)
    assert not np.array_equal(res3.groups, res.groups)


def _first_candidates(oracle, p_target, order, us):
    """Bonus tokens of all-accepted one-position sequences over singleton groups: the first candidate itself."""
    V = len(p_target)
    g = W.groups_from_lists(V, [[t] for t in range(V)])
    N = len(us)
    row = np.log(np.asarray(p_target, np.float64)).astype(np.float32)
    tl = np.broadcast_to(row, (N, 2, V)).copy()
    dl = tl[:, :1].copy()  # draft == target: every position is accepted
    u = np.zeros((N, 2, 2), np.float32)
    u[:, 1, 1] = 0.5
    tu = np.zeros((N, 2, 3), np.float32)
    tu[:, 0, 0] = np.asarray(us, np.float32)
    res = oracle.verify(tl, dl, np.zeros((N, 1), np.int32), g.group_ptr, g.group_tok, g.tok_degree, u, thin_uniforms=tu,
                        cand_order=order)
    assert np.all(res.accept_len == 1) and np.all(res.trials == 1)
    return res.tokens[:, 1].tolist()


def test_thinning_candidate_walks_the_tokens_in_the_given_order(oracle):
    """Expected tokens written out by hand.  Target p = (0.1, 0.2, 0.3, 0.4) over tokens 0..3.
    Order (2, 0, 3, 1): running sums 0.3 (token 2), 0.4 (token 0), 0.8 (token 3), 1.0 (token 1).
    Ascending order: running sums 0.1, 0.3, 0.6, 1.0."""
    p = [0.1, 0.2, 0.3, 0.4]
    us = [0.05, 0.29, 0.31, 0.39, 0.41, 0.79, 0.81, 0.99]
    assert _first_candidates(oracle, p, np.array([2, 0, 3, 1], np.int32), us) == [2, 2, 0, 0, 3, 3, 1, 1]
    assert _first_candidates(oracle, p, None, us) == [0, 1, 2, 2, 2, 3, 3, 3]
    assert _first_candidates(oracle, p, np.arange(4, dtype=np.int32), us) == [0, 1, 2, 2, 2, 3, 3, 3]
    # uniform target over eight tokens: the candidate is the floor(8 u)-th token of the order
    order = np.array([5, 2, 7, 0, 3, 6, 1, 4], np.int32)
    us8 = [(i + 0.5) / 8 for i in range(8)]
    assert _first_candidates(oracle, [0.125] * 8, order, us8) == [5, 2, 7, 0, 3, 6, 1, 4]
    assert _first_candidates(oracle, [0.125] * 8, None, us8) == [0, 1, 2, 3, 4, 5, 6, 7]


def test_thinning_rejects_an_order_that_is_no_permutation(oracle):
    for bad in ([0, 1, 1, 3], [0, 1, 2, 4], [-1, 0, 1, 2]):
        with pytest.raises(ValueError):
            _first_candidates(oracle, [0.25] * 4, np.array(bad, np.int32), [0.5])
    with pytest.raises(ValueError):
        _first_candidates(oracle, [0.25] * 4, np.arange(3, dtype=np.int32), [0.5])
