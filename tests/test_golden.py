"""The oracle must keep returning what it returned for the stored explicit case
(tests/golden/algorithm1_small.json, written by tests/golden/make_golden.py)."""
import json
import os

import numpy as np


def _case():
    with open(os.path.join(os.path.dirname(__file__), "golden", "algorithm1_small.json")) as f:
        d = json.load(f)
    d["u"] = (np.array(d["uniforms_times_2p24"], np.float64) * 2.0 ** -24).astype(np.float32)
    return d


def test_oracle_reproduces_stored_case(oracle):
    d = _case()
    res = oracle.verify(np.array(d["target_logits"], np.float32), np.array(d["draft_logits"], np.float32),
                        np.array(d["draft_tokens"], np.int32), d["group_ptr"], d["group_tok"], d["tok_degree"], d["u"],
                        d["temperature"])
    assert res.accept_len.tolist() == d["accept_len"]
    assert res.tokens.tolist() == d["tokens"]
    assert res.groups.tolist() == d["groups"]
    P = oracle.group_probs(np.array(d["target_logits"], np.float32).reshape(-1, d["V"]), d["group_ptr"],
                           d["group_tok"], d["tok_degree"], d["temperature"])
    np.testing.assert_allclose(P, np.array(d["target_group_probs"]), rtol=1e-13)
    np.testing.assert_allclose(P.sum(axis=1), 1.0, rtol=1e-13)  # Sec. 2.2: no renormalisation is needed
    assert sorted(set(d["accept_len"])) != [0]  # the stored case exercises acceptances as well as rejections
