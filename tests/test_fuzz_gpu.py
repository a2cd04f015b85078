"""Randomised shapes: every seed draws a small problem (vocabulary, groups, drafted positions, batch, element type,
membership recipe, equal split or general weights, temperature, a few masked logits) and checks all pcg_verify modes
and pcg_verify_thinning against the oracle, decision by decision."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.compare import compare_verify  # noqa: E402

from gpu_util import make_handle, run_oracle, run_verify  # noqa: E402
from test_thinning_gpu import assert_thin_parity, oracle_thin, run_thin  # noqa: E402


@pytest.mark.parametrize("seed", range(60))
def test_random_problem_matches_oracle_in_every_mode(oracle, seed):
    rng = np.random.default_rng(7000 + seed)
    V = int(rng.choice([37, 256, 999, 2048, 5000, 12000]))
    M = int(max(2, min(V, rng.choice([3, V // 20 + 2, V // 5 + 1, V // 2]))))
    K = int(rng.choice([1, 2, 5, 9, 17, 40]))
    B = int(rng.choice([1, 3, 33, 70, 140, 260]))
    if B * K * V > 3e7:  # keep the oracle's work to a second or two
        B = max(1, int(3e7 // (K * V)))
    dtype = str(rng.choice(["f32", "bf16", "f16"]))
    base = str(rng.choice(["C1", "C2", "C3", "C4"]))
    if M < 16 or V < 999:  # the threshold and heavy-tail recipes need room (8 nearest centroids, group sizes up to 200)
        base = "C1"
    cfg = W.scaled(W.CONFIGS[base], B=B, K=K, V=V, M=M, dtype=dtype, temperature=float(rng.choice([1.0, 0.8, 1.7])),
                   emb_dim=(16 if W.CONFIGS[base].emb_dim else 0), degree=int(min(M, rng.choice([1, 2, 3, 5]))))
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    if rng.random() < 0.5:  # draft close to the target: long accepted runs and bonus rows
        mix = np.float32(rng.choice([0.0, 0.1]))
        tgt = bt.target_logits[:, :K]
        if dtype == "bf16":
            t32, d32 = W.bf16_bits_to_f32(tgt), W.bf16_bits_to_f32(bt.draft_logits)
            bt.draft_logits[:] = W.f32_to_bf16_bits(t32 + mix * (d32 - t32))
        else:
            bt.draft_logits[:] = (tgt.astype(np.float32) + mix * (bt.draft_logits.astype(np.float32) - tgt.astype(np.float32))).astype(bt.draft_logits.dtype)
    weights = None
    if rng.random() < 0.4:
        raw = rng.random(groups.nnz) + 0.05
        tot = np.zeros(V)
        np.add.at(tot, groups.group_tok, raw)
        weights = (raw / tot[groups.group_tok]).astype(np.float32)
    w64 = None if weights is None else weights.astype(np.float64)
    h = make_handle(groups, weights=weights)
    ref = run_oracle(oracle, bt, groups, weights=w64)
    modes = [0, 1, 4] + ([2] if h.info.slices > 0 else [])
    for mode in modes:
        got = run_verify(bt, h, mode=mode)
        cmp = compare_verify(got[0], got[1], got[2], ref, band=1e-6)
        assert cmp.hard == 0, (seed, mode, cmp.details[:3])
        assert cmp.excused <= 1, (seed, mode, cmp.details[:3])
    tu = W.make_thin_uniforms(cfg, int(rng.choice([1, 3, 20, 50])))
    tref = oracle_thin(oracle, bt, groups, tu, weights=w64)
    assert_thin_parity(run_thin(bt, h, tu), tref, max_excused=1)
