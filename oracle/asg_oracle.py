"""Acoustic Similarity Groups from an embedding table -- CPU oracle (TEST INFRASTRUCTURE, NOT PRODUCT CODE).

The paper's group-construction equation (Sec. 2.1): the group of token t is every token whose embedding has
cosine similarity with Emb(t) strictly above a threshold theta,

    G(t) = { t' in V : cos(Emb(t), Emb(t')) > theta },

and the collection of DISTINCT sets G(t) forms the group set {G_k}, k = 1..M, M <= |V|.  This file writes that
definition out in float64 with numpy (a library matrix product is one step; no blocking beyond what memory
needs), shares nothing with the CUDA sources and is imported only by tests, the smoke check and the benchmark's
CPU leg.

Readings where the paper is silent:
  * t is always a member of G(t) (cos(x, x) = 1 > theta for any theta < 1); this is enforced also for a zero
    embedding, whose cosine is undefined, and for theta >= 1, so that every token has degree >= 1.
  * a zero embedding has cosine 0 with every other token.
  * groups are numbered in order of the smallest token t whose G(t) equals the set; tokens inside a group
    ascend; N(t) counts the distinct groups containing t.
  * embeddings given as bfloat16 bit patterns (uint16) or float32 are widened exactly; float32 tables are first
    rounded to bfloat16 (nearest even) because that is the precision the similarity is defined in for this
    library (`round_to_bf16=True`).

Parity status: pinned by tests/test_asg_oracle_pins.py (a pure-Python statement of the definition on tiny tables,
a hand-worked table with exactly known cosines, limiting thresholds, duplicated embeddings).  Agreement with the
authors' own group files is "parity unpinned": neither their embeddings nor their groups are published.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


def _bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(x, np.float32).view(np.uint32)
    return ((b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


@dataclass
class AsgResult:
    group_ptr: np.ndarray  # [M+1] int32
    group_tok: np.ndarray  # [nnz] int32, ascending inside a group
    tok_degree: np.ndarray  # [V] int32
    representative: np.ndarray  # [M] int32: smallest token whose neighbourhood is the group
    min_margin: float  # smallest |cos - theta| over all pairs t != t' (how close any decision is to flipping)

    @property
    def M(self) -> int:
        return int(self.group_ptr.shape[0] - 1)


def widen(emb, round_to_bf16: bool = True) -> np.ndarray:
    """The float64 table the similarity is defined on."""
    emb = np.asarray(emb)
    if emb.dtype == np.uint16:
        return _bf16_bits_to_f64(emb)
    if emb.dtype == np.float32:
        return _bf16_bits_to_f64(_f32_to_bf16_bits(emb)) if round_to_bf16 else emb.astype(np.float64)
    raise TypeError("embeddings must be float32 or uint16 (bf16 bit patterns)")


def neighbourhoods(emb, theta: float, round_to_bf16: bool = True, chunk: int = 1024):
    """Boolean matrix nb[t, t'] = (t' in G(t)) and the smallest |cos - theta| over t != t'."""
    E = widen(emb, round_to_bf16)
    V = E.shape[0]
    norm = np.sqrt((E * E).sum(axis=1))
    inv = np.where(norm > 0, 1.0 / np.where(norm > 0, norm, 1.0), 0.0)
    nb = np.zeros((V, V), dtype=bool)
    min_margin = np.inf
    th = float(np.float32(theta))  # the threshold is passed to the library as a float32
    for lo in range(0, V, chunk):
        hi = min(V, lo + chunk)
        cos = (E[lo:hi] @ E.T) * inv[lo:hi, None] * inv[None, :]
        nb[lo:hi] = cos > th
        m = np.abs(cos - th)
        m[np.arange(hi - lo), np.arange(lo, hi)] = np.inf  # the diagonal is not a decision
        min_margin = min(min_margin, float(m.min())) if V > 1 else min_margin
    nb[np.arange(V), np.arange(V)] = True  # t is always in G(t)
    return nb, min_margin


def build_groups(emb, theta: float, round_to_bf16: bool = True) -> AsgResult:
    """Distinct neighbourhoods as a group -> token CSR, with token degrees."""
    nb, min_margin = neighbourhoods(emb, theta, round_to_bf16)
    V = nb.shape[0]
    seen = {}
    reps = []
    for t in range(V):  # distinct sets, numbered by first appearance
        key = np.packbits(nb[t]).tobytes()
        if key not in seen:
            seen[key] = len(reps)
            reps.append(t)
    ptr = np.zeros(len(reps) + 1, np.int64)
    toks = []
    for k, t in enumerate(reps):
        members = np.nonzero(nb[t])[0]
        toks.append(members)
        ptr[k + 1] = ptr[k] + members.size
    tok = np.concatenate(toks).astype(np.int32) if toks else np.zeros(0, np.int32)
    deg = np.bincount(tok, minlength=V).astype(np.int32)
    return AsgResult(ptr.astype(np.int32), tok, deg, np.asarray(reps, np.int32), min_margin)
