"""Seeded synthetic inputs shaped like the paper's TTS verification workloads.

This module only draws inputs (logits, group memberships, drafted tokens,
uniforms).  It holds none of the verification arithmetic and imports neither
the CUDA binding nor the CPU oracle, so both can be fed from it.

The paper's real workload (LLaSA-8B logits over the 65,536-entry X-codec2
codebook, groups from the model's embedding table, LibriTTS prompts; Sec. 3.1)
is not available offline; these generators stand in for it with the same shapes
(V up to 65,536, temperature 0.8 where stated, group sizes up to ~200).

Everything is a pure function of (config name, sequence index): sequence ``b``
of a config can be regenerated alone, which is what the full-size parity checks
do.  bf16 logits are returned as uint16 bit patterns, fp16 logits as numpy float16.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Optional, Sequence

import numpy as np

SEED0 = 251113732
_STREAM_EMB, _STREAM_CENT, _STREAM_SEQ, _STREAM_GROUPS, _STREAM_THIN = 0, 1, 2, 3, 4


@dataclass(frozen=True)
class Config:
    name: str
    cfg_id: int
    B: int
    K: int
    V: int
    M: int
    dtype: str  # "f32" | "bf16" | "f16"
    temperature: float
    logits: str  # recipe name
    groups: str  # recipe name
    emb_dim: int = 0
    degree: int = 0


CONFIGS = {
    "C1": Config("C1", 1, 1, 4, 1024, 256, "f32", 1.0, "gauss2_noise1", "topk", 64, 3),
    "C2": Config("C2", 2, 16, 8, 4096, 1024, "f32", 1.0, "gauss3_boost", "threshold", 128, 3),
    "C3": Config("C3", 3, 64, 8, 8192, 2048, "bf16", 1.0, "gauss3_noise15", "topk", 256, 4),
    "C4": Config("C4", 4, 128, 12, 16384, 4096, "bf16", 0.8, "zipf_rho07", "heavy_tail", 0, 5),
    "C5": Config("C5", 5, 256, 16, 65536, 16384, "bf16", 1.0, "gauss4_mix06", "topk", 512, 6),
    # variants of C5 used as parity pins: a partition (every token in exactly one
    # group) and singleton groups (group g = {g}), both of which must reproduce
    # token-level speculative sampling.
    "C5d": Config("C5d", 5, 256, 16, 65536, 16384, "bf16", 1.0, "gauss4_mix06", "topk", 512, 1),
    "C5s": Config("C5s", 5, 256, 16, 65536, 65536, "bf16", 1.0, "gauss4_mix06", "singleton", 0, 1),
}


@dataclass
class Groups:
    """Group -> token CSR (tokens ascending inside a group) plus token degrees N(t)."""
    V: int
    M: int
    group_ptr: np.ndarray  # [M+1] int32
    group_tok: np.ndarray  # [nnz] int32
    tok_degree: np.ndarray  # [V] int32

    @property
    def nnz(self) -> int:
        return int(self.group_ptr[-1])


@dataclass
class Batch:
    target_logits: np.ndarray  # [B, K+1, V] float32 or uint16 (bf16 bits)
    draft_logits: np.ndarray  # [B, K, V]
    draft_tokens: np.ndarray  # [B, K] int32
    uniforms: np.ndarray  # [B, K+1, 2] float32, multiples of 2^-24 in [0, 1)
    temperature: float
    dtype: str


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even) and return the 16-bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(cfg_id: int, stream: int, index: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([SEED0, cfg_id, stream, index])))


def groups_from_lists(V: int, lists: Sequence[Sequence[int]]) -> Groups:
    """Build the CSR and the degree array from explicit token lists (one per group)."""
    ptr = np.zeros(len(lists) + 1, np.int32)
    toks = []
    for g, lst in enumerate(lists):
        s = sorted(int(t) for t in lst)
        toks.extend(s)
        ptr[g + 1] = len(toks)
    tok = np.asarray(toks, np.int32).reshape(-1)
    deg = np.bincount(tok, minlength=V).astype(np.int32) if tok.size else np.zeros(V, np.int32)
    return Groups(V, len(lists), ptr, tok, deg)


def _csr_from_pairs(V: int, M: int, g: np.ndarray, t: np.ndarray) -> Groups:
    order = np.lexsort((t, g))
    g, t = g[order], t[order]
    ptr = np.zeros(M + 1, np.int64)
    np.add.at(ptr, g + 1, 1)
    ptr = np.cumsum(ptr).astype(np.int32)
    deg = np.bincount(t, minlength=V).astype(np.int32)
    return Groups(V, M, ptr, t.astype(np.int32), deg)


def _embeddings(cfg: Config):
    """Seeded unit-norm Gaussian token embeddings [V, d] and the centroid matrix [d, M] (M distinct tokens)."""
    emb = _rng(cfg.cfg_id, _STREAM_EMB).standard_normal((cfg.V, cfg.emb_dim), dtype=np.float32)
    emb /= np.linalg.norm(emb, axis=1, keepdims=True)
    cent_ids = _rng(cfg.cfg_id, _STREAM_CENT).permutation(cfg.V)[: cfg.M]
    return emb, np.ascontiguousarray(emb[cent_ids].T)


def _nearest_centroids(cfg: Config, k: int, chunk: int = 2048, threads: int = 8):
    """Per token, the k centroids of largest cosine, best first: (ids [V,k], cosines [V,k])."""
    emb, cent = _embeddings(cfg)
    ids = np.empty((cfg.V, k), np.int64)
    cosv = np.empty((cfg.V, k), np.float32)

    def work(lo):
        hi = min(cfg.V, lo + chunk)
        cos = emb[lo:hi] @ cent
        if k == 1:
            idx = np.argmax(cos, axis=1)[:, None]
        else:
            idx = np.argpartition(-cos, k - 1, axis=1)[:, :k]
        c = np.take_along_axis(cos, idx, axis=1)
        o = np.argsort(-c, axis=1, kind="stable")
        ids[lo:hi] = np.take_along_axis(idx, o, axis=1)
        cosv[lo:hi] = np.take_along_axis(c, o, axis=1)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(work, range(0, cfg.V, chunk)))
    return ids, cosv


def _groups_topk(cfg: Config) -> Groups:
    k = cfg.degree
    ids, _ = _nearest_centroids(cfg, k)
    return _csr_from_pairs(cfg.V, cfg.M, ids.reshape(-1), np.repeat(np.arange(cfg.V), k))


def _groups_threshold(cfg: Config, dmax: int = 8) -> Groups:
    """Membership = centroids with cosine above a threshold tuned for the mean degree,
    clamped to [1, dmax] per token (always the nearest centroid, at most the dmax nearest)."""
    top_idx, top_cos = _nearest_centroids(cfg, dmax)

    def mean_degree(theta):
        return np.maximum(1, (top_cos > theta).sum(axis=1)).mean()

    lo_t, hi_t = -1.0, 1.0
    for _ in range(40):  # bisection on the threshold
        mid = 0.5 * (lo_t + hi_t)
        if mean_degree(mid) > cfg.degree:
            lo_t = mid
        else:
            hi_t = mid
    keep = top_cos > hi_t
    keep[:, 0] = True
    t = np.repeat(np.arange(cfg.V), dmax).reshape(cfg.V, dmax)
    return _csr_from_pairs(cfg.V, cfg.M, top_idx[keep], t[keep])


def _groups_heavy_tail(cfg: Config, dmax: int = 16, smax: int = 200) -> Groups:
    """Configuration-model bipartite graph: token degrees from a truncated geometric law
    (mean ~cfg.degree), group sizes from a truncated Pareto law in [1, smax]."""
    rng = _rng(cfg.cfg_id, _STREAM_GROUPS)
    deg = np.minimum(dmax, rng.geometric(1.0 / cfg.degree, size=cfg.V)).astype(np.int64)
    nnz = int(deg.sum())
    raw = (1.0 - rng.random(cfg.M)) ** (-1.0 / 1.3)
    lo_s, hi_s = 0.0, float(smax)
    for _ in range(60):  # bisection on the scale so that the clipped sizes sum to ~nnz
        mid = 0.5 * (lo_s + hi_s)
        if np.clip(np.rint(1.0 + (raw - 1.0) * mid), 1, smax).sum() < nnz:
            lo_s = mid
        else:
            hi_s = mid
    size = np.clip(np.rint(1.0 + (raw - 1.0) * hi_s), 1, smax).astype(np.int64)
    while size.sum() != nnz:  # spread the rounding remainder over distinct random groups
        diff = int(nnz - size.sum())
        step = 1 if diff > 0 else -1
        idx = rng.permutation(cfg.M)
        idx = idx[(size[idx] + step >= 1) & (size[idx] + step <= smax)][: abs(diff)]
        size[idx] += step
    stubs = np.repeat(np.arange(cfg.V), deg)
    rng.shuffle(stubs)
    slot_group = np.repeat(np.arange(cfg.M), size)
    for _ in range(200):  # resolve duplicate (group, token) pairs by swapping stubs
        key = slot_group * cfg.V + stubs
        order = np.argsort(key, kind="stable")
        dup = order[1:][key[order][1:] == key[order][:-1]]
        if dup.size == 0:
            break
        partner = rng.integers(0, nnz, size=dup.size)
        stubs[dup], stubs[partner] = stubs[partner].copy(), stubs[dup].copy()
    else:
        raise RuntimeError("could not resolve duplicate memberships")
    # overlapping swaps can, at small sizes, take a token's last stub away: every token must be in a group
    missing = np.setdiff1d(np.arange(cfg.V), stubs)
    if missing.size:
        slot_group = np.concatenate([slot_group, missing % cfg.M])
        stubs = np.concatenate([stubs, missing])
    return _csr_from_pairs(cfg.V, cfg.M, slot_group, stubs)


_GROUP_CACHE: dict = {}


def make_groups(cfg: Config) -> Groups:
    key = (cfg.cfg_id, cfg.V, cfg.M, cfg.groups, cfg.emb_dim, cfg.degree)
    if key not in _GROUP_CACHE:
        if cfg.groups == "topk":
            g = _groups_topk(cfg)
        elif cfg.groups == "threshold":
            g = _groups_threshold(cfg)
        elif cfg.groups == "heavy_tail":
            g = _groups_heavy_tail(cfg)
        elif cfg.groups == "singleton":
            g = Groups(cfg.V, cfg.V, np.arange(cfg.V + 1, dtype=np.int32), np.arange(cfg.V, dtype=np.int32),
                       np.ones(cfg.V, np.int32))
        else:
            raise ValueError(cfg.groups)
        _GROUP_CACHE[key] = g
    return _GROUP_CACHE[key]


def _logit_rows(cfg: Config, rng: np.random.Generator):
    """float32 target [K+1, V] and draft [K, V] logits of one sequence, before any bf16 rounding."""
    K, V = cfg.K, cfg.V
    n = rng.standard_normal
    if cfg.logits == "gauss2_noise1":
        tgt = 2.0 * n((K + 1, V), dtype=np.float32)
        drf = tgt[:K] + n((K, V), dtype=np.float32)
    elif cfg.logits == "gauss3_boost":
        tgt = 3.0 * n((K + 1, V), dtype=np.float32)
        nb = max(1, V // 100)
        for r in range(K + 1):
            tgt[r, rng.choice(V, size=nb, replace=False)] += 6.0
        drf = 0.8 * tgt[:K] + n((K, V), dtype=np.float32)
    elif cfg.logits == "gauss3_noise15":
        tgt = 3.0 * n((K + 1, V), dtype=np.float32)
        drf = tgt[:K] + 1.5 * n((K, V), dtype=np.float32)
    elif cfg.logits == "zipf_rho07":
        base = (-1.2 * np.log(np.arange(1, V + 1, dtype=np.float64))).astype(np.float32)
        tgt = np.empty((K + 1, V), np.float32)
        for r in range(K + 1):
            tgt[r] = base[rng.permutation(V)]
        tgt += 0.5 * n((K + 1, V), dtype=np.float32)
        mu = tgt[:K].mean(axis=1, keepdims=True)
        sd = tgt[:K].std(axis=1, keepdims=True)
        z = (tgt[:K] - mu) / sd
        drf = mu + sd * (0.7 * z + np.float32(np.sqrt(1.0 - 0.49)) * n((K, V), dtype=np.float32))
    elif cfg.logits == "gauss4_mix06":
        tgt = 4.0 * n((K + 1, V), dtype=np.float32)
        drf = 0.6 * tgt[:K] + 2.0 * n((K, V), dtype=np.float32)
    else:
        raise ValueError(cfg.logits)
    return tgt.astype(np.float32), drf.astype(np.float32)


def make_sequence(cfg: Config, b: int):
    """Inputs of sequence b: (target [K+1,V], draft [K,V], draft_tokens [K], uniforms [K+1,2])."""
    rng = _rng(cfg.cfg_id, _STREAM_SEQ, b)
    tgt, drf = _logit_rows(cfg, rng)
    if cfg.dtype == "bf16":
        tgt_s, drf_s = f32_to_bf16_bits(tgt), f32_to_bf16_bits(drf)
        drf_val = bf16_bits_to_f32(drf_s)
    elif cfg.dtype == "f16":
        tgt_s, drf_s = tgt.astype(np.float16), drf.astype(np.float16)
        drf_val = drf_s.astype(np.float32)
    else:
        tgt_s, drf_s, drf_val = tgt, drf, drf
    # drafted tokens follow the draft distribution at the call's temperature; drawn with
    # the Gumbel-max trick so that no normalised distribution is formed here
    gumbel = -np.log(-np.log(rng.random((cfg.K, cfg.V), dtype=np.float32) + np.float32(1e-30)))
    tokens = np.argmax(drf_val / np.float32(cfg.temperature) + gumbel, axis=1).astype(np.int32)
    uniforms = (rng.integers(0, 1 << 24, size=(cfg.K + 1, 2)).astype(np.float32) * np.float32(2.0 ** -24))
    return tgt_s, drf_s, tokens, uniforms


def make_batch(cfg: Config, B: Optional[int] = None, seqs: Optional[Sequence[int]] = None, threads: int = 8) -> Batch:
    """Stack sequences 0..B-1 (or the listed ones) of a config into one batch."""
    if seqs is None:
        seqs = range(cfg.B if B is None else B)
    seqs = list(seqs)
    dt = {"bf16": np.uint16, "f16": np.float16}.get(cfg.dtype, np.float32)
    n = len(seqs)
    tl = np.empty((n, cfg.K + 1, cfg.V), dt)
    dl = np.empty((n, cfg.K, cfg.V), dt)
    x = np.empty((n, cfg.K), np.int32)
    u = np.empty((n, cfg.K + 1, 2), np.float32)

    def fill(i):
        tl[i], dl[i], x[i], u[i] = make_sequence(cfg, seqs[i])

    if n > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(n)))
    else:
        for i in range(n):
            fill(i)
    return Batch(tl, dl, x, u, cfg.temperature, cfg.dtype)


def make_thin_uniforms(cfg: Config, n_trials: int, B: Optional[int] = None, seqs: Optional[Sequence[int]] = None) -> np.ndarray:
    """Uniforms of the thinning trials, [n, n_trials, 3] float32 multiples of 2^-24 in [0, 1): per trial the
    token, label and keep draw.  A pure function of (config, sequence index), like the other inputs."""
    if seqs is None:
        seqs = range(cfg.B if B is None else B)
    seqs = list(seqs)
    out = np.empty((len(seqs), n_trials, 3), np.float32)
    for i, b in enumerate(seqs):
        rng = _rng(cfg.cfg_id, _STREAM_THIN, b)
        out[i] = rng.integers(0, 1 << 24, size=(n_trials, 3)).astype(np.float32) * np.float32(2.0 ** -24)
    return out


def scaled(cfg: Config, **kw) -> Config:
    """A copy of a config with some sizes overridden (for small parity cases)."""
    return replace(cfg, **kw)
