"""Pins for the group-construction oracle (oracle/asg_oracle.py): a hand-worked table with exactly known
cosines, a loop-by-loop restatement of the definition on tiny tables, limiting thresholds and structural facts.
None of the expected values comes from the oracle itself."""
import math

import numpy as np
import pytest

from oracle import asg_oracle as A
from paper_2511_13732_b200 import workloads as W


def _lists(res):
    return [res.group_tok[res.group_ptr[k]:res.group_ptr[k + 1]].tolist() for k in range(res.M)]


# Table: e1, 2*e1 (same direction), e2, e1+e2 (45 degrees: cosine 1/sqrt(2) = 0.7071 with e1 and e2), zero vector.
HAND = np.array([[1, 0], [2, 0], [0, 1], [1, 1], [0, 0]], np.float32)


def test_hand_worked_table():
    r = A.build_groups(HAND, 0.5)
    # G(0) = G(1) = {0,1,3}; G(2) = {2,3}; G(3) = {0,1,2,3}; the zero vector is similar to nothing but itself
    assert _lists(r) == [[0, 1, 3], [2, 3], [0, 1, 2, 3], [4]]
    assert r.representative.tolist() == [0, 2, 3, 4]
    assert r.tok_degree.tolist() == [2, 2, 2, 3, 1]
    assert abs(r.min_margin - (1 / math.sqrt(2) - 0.5)) < 1e-12
    r = A.build_groups(HAND, 0.8)  # 0.7071 is now below the threshold
    assert _lists(r) == [[0, 1], [2], [3], [4]] and r.tok_degree.tolist() == [1, 1, 1, 1, 1]


def test_threshold_is_strict():
    # the 45-degree pair has cosine fl(1/sqrt(2)) in double; a threshold equal to the float32 value just above
    # excludes it, the float32 value just below includes it
    c = 1 / math.sqrt(2)
    above, below = np.nextafter(np.float32(c), np.float32(1)), np.nextafter(np.float32(c), np.float32(0))
    assert _lists(A.build_groups(HAND, float(above)))[0] == [0, 1]
    assert _lists(A.build_groups(HAND, float(below)))[0] == [0, 1, 3]


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_matches_the_definition_written_as_loops(seed):
    rng = np.random.default_rng(seed)
    V, d, theta = 14, 5, 0.25
    emb = W.bf16_bits_to_f32(W.f32_to_bf16_bits(rng.standard_normal((V, d)).astype(np.float32)))
    emb[5] = 3 * emb[2]  # same direction: identical neighbourhoods, merged into one group
    emb = W.bf16_bits_to_f32(W.f32_to_bf16_bits(emb))
    sets = []
    for t in range(V):
        members = []
        for u in range(V):
            dot = sum(float(emb[t, k]) * float(emb[u, k]) for k in range(d))
            nt = math.sqrt(sum(float(emb[t, k]) ** 2 for k in range(d)))
            nu = math.sqrt(sum(float(emb[u, k]) ** 2 for k in range(d)))
            if u == t or dot / (nt * nu) > float(np.float32(theta)):
                members.append(u)
        sets.append(members)
    distinct = []
    for s in sets:
        if s not in distinct:
            distinct.append(s)
    r = A.build_groups(emb, theta)
    assert _lists(r) == distinct
    assert sets[5] == sets[2] and len(distinct) < V
    want_deg = [sum(t in s for s in distinct) for t in range(V)]
    assert r.tok_degree.tolist() == want_deg


def test_limiting_thresholds_and_structure():
    rng = np.random.default_rng(7)
    emb = rng.standard_normal((40, 8)).astype(np.float32)
    one = A.build_groups(emb, -1.5)  # every pair is similar: a single group of all tokens
    assert one.M == 1 and _lists(one) == [list(range(40))] and np.all(one.tok_degree == 1)
    single = A.build_groups(emb, 1.5)  # nothing is similar: singletons, in token order
    assert single.M == 40 and _lists(single) == [[t] for t in range(40)]
    mid = A.build_groups(emb, 0.2)
    nb, _ = A.neighbourhoods(emb, 0.2)
    assert np.array_equal(nb, nb.T) and np.all(np.diag(nb))  # cosine is symmetric; t is in G(t)
    assert mid.tok_degree.sum() == mid.group_tok.size and np.all(mid.tok_degree >= 1)
    for k, t in enumerate(mid.representative):  # the group numbered k is the neighbourhood of its representative
        assert _lists(mid)[k] == np.nonzero(nb[t])[0].tolist()
    assert np.all(np.diff(mid.representative) > 0)


def test_float32_tables_are_rounded_to_bfloat16_first():
    rng = np.random.default_rng(9)
    emb = rng.standard_normal((30, 6)).astype(np.float32)
    bits = W.f32_to_bf16_bits(emb)
    a, b = A.build_groups(emb, 0.3), A.build_groups(bits, 0.3)
    assert np.array_equal(a.group_ptr, b.group_ptr) and np.array_equal(a.group_tok, b.group_tok)
    np.testing.assert_array_equal(A.widen(emb), W.bf16_bits_to_f32(bits).astype(np.float64))
