"""The per-sequence status bits on inputs that trigger them (all host-made, ordinary floating-point data; nothing
here faults): PCG_FLAG_NONFINITE for rows with a NaN, a +inf or nothing but -inf, and PCG_FLAG_ZERO_RESIDUAL for a
rejection whose residual sums to zero in float32.  Every mode of pcg_verify and pcg_verify_thinning: the flag is
set on the affected sequences and only there, every output is in range, the other sequences still match the
oracle, and the call returns."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.compare import compare_verify  # noqa: E402

from gpu_util import library_candidate_order, logits_to_device, make_handle, run_oracle, run_verify  # noqa: E402

NONFINITE, ZERO_RESIDUAL, EXHAUSTED = 4, 2, 8
MODES = [pytest.param(0, id="default"), pytest.param(1, id="dense"), pytest.param(2, id="cluster"),
         pytest.param(4, id="batched")]


def _thin(bt, handle, tu):
    from paper_2511_13732_b200 import binding

    out = binding.pcg_verify_thinning(logits_to_device(bt.target_logits), logits_to_device(bt.draft_logits),
                                      torch.from_numpy(bt.draft_tokens).cuda(), handle, torch.from_numpy(bt.uniforms).cuda(),
                                      torch.from_numpy(tu).cuda(), bt.temperature)
    torch.cuda.synchronize()
    return tuple(o.cpu().numpy() for o in out)


def _poisoned(dtype):
    """A small batch whose sequences 1..5 carry, at drafted position 0: a NaN in the target row, a +inf in the target
    row, a target row of -inf only, a draft row of -inf only, a NaN in the draft row."""
    cfg = W.scaled(W.CONFIGS["C3"], B=12, K=5, V=3000, M=500, emb_dim=16)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    if dtype == "f32":
        tl, dl = W.bf16_bits_to_f32(bt.target_logits), W.bf16_bits_to_f32(bt.draft_logits)
    else:
        tl, dl = bt.target_logits.copy(), bt.draft_logits.copy()
    nan, pinf, ninf = (np.float32(np.nan), np.float32(np.inf), np.float32(-np.inf)) if dtype == "f32" else (
        np.uint16(0x7FC0), np.uint16(0x7F80), np.uint16(0xFF80))
    tl[1, 0, 1234] = nan
    tl[2, 0, 77] = pinf
    tl[3, 0, :] = ninf
    dl[4, 0, :] = ninf
    dl[5, 0, 2999] = nan
    bad = [1, 2, 3, 4, 5]
    return cfg, groups, W.Batch(tl, dl, bt.draft_tokens, bt.uniforms, bt.temperature, dtype), bad


def _check_outputs_in_range(cfg, groups, n, tok, grp):
    assert np.all((n >= 0) & (n <= cfg.K))
    assert np.all((tok >= -1) & (tok < cfg.V)) and np.all((grp >= -1) & (grp < groups.M))
    for b in range(cfg.B):
        assert np.all(tok[b, :n[b] + 1] >= 0) and np.all(tok[b, n[b] + 1:] == -1)
        assert np.all(grp[b, :n[b] + 1] >= 0) and np.all(grp[b, n[b] + 1:] == -1)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_nonfinite_rows_are_flagged_and_harmless(oracle, dtype, mode):
    cfg, groups, bt, bad = _poisoned(dtype)
    h = make_handle(groups)
    n, tok, grp, flg = run_verify(bt, h, mode=mode)
    _check_outputs_in_range(cfg, groups, n, tok, grp)
    good = [b for b in range(cfg.B) if b not in bad]
    assert np.all(flg[bad] & NONFINITE), flg
    assert np.all(flg[good] == 0), flg
    # the clean sequences are untouched by their neighbours
    sub = W.Batch(bt.target_logits[good], bt.draft_logits[good], bt.draft_tokens[good], bt.uniforms[good], bt.temperature,
                  bt.dtype)
    cmp = compare_verify(n[good], tok[good], grp[good], run_oracle(oracle, sub, groups))
    assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]
    # bit-reproducible also on such rows
    again = run_verify(bt, h, mode=mode)
    assert all(np.array_equal(a, b) for a, b in zip((n, tok, grp, flg), again))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_nonfinite_rows_in_the_thinning_entry_point(oracle, dtype):
    cfg, groups, bt, bad = _poisoned(dtype)
    h = make_handle(groups)
    tu = W.make_thin_uniforms(cfg, 6)
    n, tok, grp, flg, trials = _thin(bt, h, tu)
    _check_outputs_in_range(cfg, groups, n, tok, grp)
    good = [b for b in range(cfg.B) if b not in bad]
    assert np.all(flg[bad] & NONFINITE), flg
    assert np.all((flg[good] & NONFINITE) == 0), flg
    assert np.all((trials >= 0) & (trials <= 6))
    sub = W.Batch(bt.target_logits[good], bt.draft_logits[good], bt.draft_tokens[good], bt.uniforms[good], bt.temperature,
                  bt.dtype)
    ref = oracle.verify(sub.target_logits, sub.draft_logits, sub.draft_tokens, groups.group_ptr, groups.group_tok,
                        groups.tok_degree, sub.uniforms, sub.temperature, threads=0, thin_uniforms=tu[good],
                        cand_order=library_candidate_order(groups.V, sub.target_logits))
    cmp = compare_verify(n[good], tok[good], grp[good], ref)
    assert cmp.hard == 0 and cmp.excused <= 1, cmp.details[:3]


def _vanishing_residual():
    """float32 rows over a partition into groups of eight tokens.  Group 0 holds tokens of negligible mass; the
    draft equals the target except that token 0 (the heaviest of group 0, about e^-30 of the row's mass) has its
    logit raised by 0.01.  The label group's draft mass is then 1 % above its target mass, so an accept uniform of
    0.995 rejects -- yet the normalisers of the two rows are the same number (the change is 1e-18 of the sum, below
    even double precision) and every other token's p - q is exactly zero, so the residual sums to zero, in the
    library and in the oracle alike.  Both then draw from the target's coarse distribution and flag the sequence
    (in exact arithmetic the residual is spread like that distribution, up to the negligible group 0)."""
    rng = np.random.default_rng(9)
    V, G8, B, K = 512, 64, 6, 3
    groups = W.groups_from_lists(V, [list(range(8 * g, 8 * g + 8)) for g in range(G8)])
    tl = rng.standard_normal((B, K + 1, V)).astype(np.float32)
    dl = tl[:, :K].copy()
    x = rng.integers(8, V, size=(B, K)).astype(np.int32)
    u = (rng.integers(0, 1 << 24, size=(B, K + 1, 2)) * 2.0 ** -24).astype(np.float32)
    u[:, :K, 1] = 0.0  # draft == target elsewhere: accept
    hit = [(1, 0), (2, 2), (4, 1)]  # (sequence, position) of the vanishing-residual rejection
    for b, i in hit:
        tl[b, i, :8] = np.array([-30, -60, -61, -62, -63, -64, -65, -66], np.float32)
        dl[b, i, :8] = tl[b, i, :8]
        dl[b, i, 0] += np.float32(0.01)
        x[b, i] = 0
        u[b, i, 1] = 0.995
    return groups, W.Batch(tl, dl, x, u, 1.0, "f32"), hit


@pytest.mark.parametrize("mode", MODES)
def test_vanishing_residual_falls_back_to_the_target_and_is_flagged(oracle, mode):
    groups, bt, hit = _vanishing_residual()
    h = make_handle(groups)
    n, tok, grp, flg = run_verify(bt, h, mode=mode)
    ref = run_oracle(oracle, bt, groups)
    assert [int(ref.accept_len[b]) for b, _ in hit] == [i for _, i in hit]  # the oracle rejects there too ...
    assert all(ref.flags[b] == ZERO_RESIDUAL for b, _ in hit)  # ... and finds no residual mass either
    cmp = compare_verify(n, tok, grp, ref)
    assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]
    hit_b = [b for b, _ in hit]
    assert np.all(flg[hit_b] == ZERO_RESIDUAL), flg
    assert np.all(np.delete(flg, hit_b) == 0), flg


def test_vanishing_residual_in_the_thinning_entry_point(oracle):
    groups, bt, hit = _vanishing_residual()
    h = make_handle(groups)
    tu = (np.random.default_rng(10).integers(0, 1 << 24, size=(bt.draft_tokens.shape[0], 3, 3)) * 2.0 ** -24).astype(np.float32)
    n, tok, grp, flg, trials = _thin(bt, h, tu)
    ref = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                        groups.tok_degree, bt.uniforms, bt.temperature, threads=0, thin_uniforms=tu,
                        cand_order=library_candidate_order(groups.V, bt.target_logits))
    cmp = compare_verify(n, tok, grp, ref)
    assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]
    hit_b = [b for b, _ in hit]
    # no candidate can be kept (no group has target mass above its draft mass in float32): every trial is used up,
    # the enumerated residual is empty too, and the draw comes from the target's coarse distribution
    assert np.all(flg[hit_b] == (ZERO_RESIDUAL | EXHAUSTED)), flg
    assert np.all(trials[hit_b] == 3)
    assert np.all(np.delete(flg, hit_b) == 0), flg


def test_hundred_repeats_are_bit_identical(oracle):
    """Same inputs, same outputs, bit for bit, a hundred times over (every mode, and the thinning entry point)."""
    cfg = W.scaled(W.CONFIGS["C4"], B=48, K=6, V=6000, M=1200)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    tu = W.make_thin_uniforms(cfg, 8)
    for mode in (0, 1, 2, 4):
        first = run_verify(bt, h, mode=mode)
        for _ in range(100 if mode in (0, 4) else 20):
            again = run_verify(bt, h, mode=mode)
            assert all(np.array_equal(a, b) for a, b in zip(first, again))
    first = _thin(bt, h, tu)
    for _ in range(100):
        again = _thin(bt, h, tu)
        assert all(np.array_equal(a, b) for a, b in zip(first, again))
