"""Writes tests/golden/algorithm1_small.json: a small, explicit verification case
(inputs spelled out in full) together with what the CPU oracle returns for it.

The paper prints no worked numeric example (its toy figure survives only as an
image), so this file is a regression fixture for the oracle's reading of
Algorithm 1, not a value taken from the paper.  It calls only ``oracle/``.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402


def main():
    rng = np.random.default_rng(20251113)
    B, K, V = 6, 3, 12
    lists = [[0, 1, 2, 3], [3, 4, 5], [5, 6, 7, 8, 9], [9, 10], [10, 11, 0], [2, 6, 11], []]
    ptr = np.cumsum([0] + [len(s) for s in lists]).astype(np.int32)
    tok = np.array([t for s in lists for t in sorted(s)], np.int32)
    deg = np.bincount(tok, minlength=V).astype(np.int32)
    # logits on a 1/8 grid so that they are exact in float32 and in bf16
    tl = (np.round(rng.normal(0, 2, (B, K + 1, V)) * 8) / 8).astype(np.float32)
    dl = (np.round((tl[:, :K] + rng.normal(0, 1, (B, K, V))) * 8) / 8).astype(np.float32)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, (B, K + 1, 2)) * 2.0 ** -24).astype(np.float32)
    T = 0.8
    res = oracle.verify(tl, dl, x, ptr, tok, deg, u, T)
    P = oracle.group_probs(tl.reshape(-1, V), ptr, tok, deg, T)
    out = {
        "what": "oracle output for an explicit small case of Algorithm 1 (group-level verification)",
        "V": V, "K": K, "B": B, "temperature": T,
        "group_ptr": ptr.tolist(), "group_tok": tok.tolist(), "tok_degree": deg.tolist(),
        "target_logits": tl.tolist(), "draft_logits": dl.tolist(), "draft_tokens": x.tolist(),
        "uniforms_times_2p24": (u.astype(np.float64) * 2 ** 24).astype(np.int64).tolist(),
        "accept_len": res.accept_len.tolist(), "tokens": res.tokens.tolist(), "groups": res.groups.tolist(),
        "target_group_probs": [[float(f"{v:.15e}") for v in row] for row in P],
    }
    with open(os.path.join(HERE, "algorithm1_small.json"), "w") as f:
        json.dump(out, f, indent=1)


if __name__ == "__main__":
    main()
