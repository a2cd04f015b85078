"""Decision-by-decision comparison of a verification result with the oracle's
(test infrastructure, not product code).

The library's outputs must equal the oracle's exactly, except where the uniform
of the FIRST differing decision of a sequence lies within ``band`` of that
decision's threshold (the oracle reports that distance as a margin).  Such
sequences are counted as excused; every other difference is hard.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass
class Comparison:
    sequences: int
    hard: int = 0
    excused: int = 0
    details: list = field(default_factory=list)  # (b, decision name, position, margin)

    @property
    def ok(self) -> bool:
        return self.hard == 0


def compare_verify(accept_len, tokens, groups, ref, band: float = 1e-6) -> Comparison:
    """Compare library outputs (numpy int arrays; groups may be None) with an OracleResult."""
    accept_len = np.asarray(accept_len)
    tokens = np.asarray(tokens)
    B, K1 = ref.tokens.shape
    K = K1 - 1
    out = Comparison(sequences=B)
    for b in range(B):
        same = accept_len[b] == ref.accept_len[b] and np.array_equal(tokens[b], ref.tokens[b])
        if same and groups is not None:
            same = np.array_equal(np.asarray(groups)[b], ref.groups[b])
        if same:
            continue
        # locate the first decision, in the order the algorithm takes them, that differs
        n_ref, n_got = int(ref.accept_len[b]), int(accept_len[b])
        first = None
        m = min(n_ref, n_got)
        if groups is not None:
            for i in range(m):  # labels of positions both sides accepted
                if np.asarray(groups)[b, i] != ref.groups[b, i]:
                    first = ("label", i, ref.margins[b, i, 0])
                    break
        if first is None and n_ref != n_got:  # one side accepted position m, the other rejected it
            first = ("accept", m, ref.margins[b, m, 1])
        if first is None:
            n = n_ref
            if groups is not None and np.asarray(groups)[b, n] != ref.groups[b, n]:
                first = ("terminal_group", n, ref.margins[b, K, 0])
            elif groups is None and tokens[b, n] != ref.tokens[b, n]:
                # without group ids the terminal group and token draws cannot be told apart
                first = ("terminal", n, min(ref.margins[b, K, 0], ref.margins[b, K, 1]))
            elif tokens[b, n] != ref.tokens[b, n]:
                first = ("terminal_token", n, ref.margins[b, K, 1])
            else:
                first = ("layout", -1, np.inf)  # same decisions, different filler or accepted tokens
        name, pos, margin = first
        if margin < band:
            out.excused += 1
        else:
            out.hard += 1
        out.details.append((b, name, pos, float(margin)))
    return out
