"""GPU parity of pcg_verify_thinning (terminal group by the paper's thinning sampler, Sec. 2.2) against the CPU
oracle's thinning sampler on the same seeded inputs and the same trial uniforms.  Accept lengths, group ids,
tokens, trial counts and flags must be identical except where the first differing decision's uniform lies within
1e-6 of its threshold (the oracle's margin of the terminal group is the smallest one over the trials it ran)."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.compare import compare_verify  # noqa: E402

from gpu_util import library_candidate_order, logits_to_device, make_handle  # noqa: E402

BAND = 1e-6
EXHAUSTED = 8


def run_thin(batch, handle, tu, **kw):
    from paper_2511_13732_b200 import binding

    tl, dl = logits_to_device(batch.target_logits), logits_to_device(batch.draft_logits)
    x = torch.from_numpy(batch.draft_tokens).cuda()
    u = torch.from_numpy(batch.uniforms).cuda()
    out = binding.pcg_verify_thinning(tl, dl, x, handle, u, torch.from_numpy(tu).cuda(), batch.temperature, **kw)
    torch.cuda.synchronize()
    return tuple(o.cpu().numpy() for o in out)


def oracle_thin(oracle, batch, groups, tu, weights=None):
    return oracle.verify(batch.target_logits, batch.draft_logits, batch.draft_tokens, groups.group_ptr,
                         groups.group_tok, groups.tok_degree, batch.uniforms, batch.temperature, weights=weights,
                         threads=0, thin_uniforms=tu,
                         cand_order=library_candidate_order(groups.V, batch.target_logits))


def assert_thin_parity(got, ref, max_excused=0):
    n, tok, grp, flg, trials = got
    cmp = compare_verify(n, tok, grp, ref, band=BAND)
    assert cmp.hard == 0, f"hard mismatches: {cmp.details[:5]}"
    assert cmp.excused <= max_excused, f"excused mismatches: {cmp.details[:5]}"
    excused = {d[0] for d in cmp.details}
    K = ref.tokens.shape[1] - 1
    quiet = 0  # same outputs reached over a different number of trials: a keep test on its threshold
    for b in range(len(n)):
        if b in excused:
            continue
        if trials[b] != ref.trials[b] or flg[b] != ref.flags[b]:
            # with few groups a later candidate can land on the same group (and then the same token): only a
            # decision within the band of its threshold may make the trial counts differ
            assert ref.margins[b, K, 0] < BAND, (b, trials[b], ref.trials[b], flg[b], ref.flags[b], ref.margins[b, K, 0])
            quiet += 1
    assert cmp.excused + quiet <= max_excused, (cmp.excused, quiet)
    return cmp


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4"])
def test_thinning_matches_oracle_on_configs(oracle, name):
    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    tu = W.make_thin_uniforms(cfg, 32)
    ref = oracle_thin(oracle, bt, groups, tu)
    got = run_thin(bt, make_handle(groups), tu)
    assert_thin_parity(got, ref)
    if cfg.B >= 16:
        assert ref.trials.max() > 1 and ref.trials.min() == 1


@pytest.mark.parametrize("name,B", [("C5", 12), ("C5d", 10)])
def test_thinning_c5_shape_small_batch(oracle, name, B):
    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=B)
    tu = W.make_thin_uniforms(cfg, 48, B=B)
    ref = oracle_thin(oracle, bt, groups, tu)
    assert_thin_parity(run_thin(bt, make_handle(groups), tu), ref)


def test_thinning_without_a_sweep_layout_singleton_groups(oracle):
    """65,536 singleton groups: token-level speculative sampling with the thinning sampler, on a handle that has
    no token-sliced layout."""
    cfg = W.CONFIGS["C5s"]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=6)
    tu = W.make_thin_uniforms(cfg, 64, B=6)
    ref = oracle_thin(oracle, bt, groups, tu)
    got = run_thin(bt, make_handle(groups), tu)
    assert_thin_parity(got, ref)
    n, tok, grp = got[0], got[1], got[2]
    assert all(tok[b, n[b]] == grp[b, n[b]] for b in range(6))


@pytest.mark.parametrize("V,dtype", [(1003, "f32"), (1003, "bf16"), (77, "bf16"), (4096 + 8, "bf16"), (5, "f32")])
def test_thinning_ragged_and_misaligned_rows(oracle, V, dtype):
    cfg = W.scaled(W.CONFIGS["C1"], B=24, K=3, V=V, M=max(2, V // 6), emb_dim=8, dtype=dtype,
                   degree=min(3, max(2, V // 6)))
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    tu = W.make_thin_uniforms(cfg, 40)
    ref = oracle_thin(oracle, bt, groups, tu)
    assert_thin_parity(run_thin(bt, make_handle(groups), tu), ref)


@pytest.mark.parametrize("K", [1, 33, 100])
def test_thinning_long_accepts_small_tv_and_bonus(oracle, K):
    """Draft close to the target: long accepted runs (bonus draws), rare rejections with a small TV, so that the
    trials go past one round of warps and some sequences run out of the 40 supplied trials."""
    cfg = W.scaled(W.CONFIGS["C1"], B=48, K=K, V=512, M=100, emb_dim=8)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    bt.draft_logits[:] = bt.target_logits[:, :K] + 0.05 * (bt.draft_logits - bt.target_logits[:, :K])
    tu = W.make_thin_uniforms(cfg, 40)
    ref = oracle_thin(oracle, bt, groups, tu)
    got = run_thin(bt, make_handle(groups), tu)
    assert_thin_parity(got, ref, max_excused=1)
    if K >= 33:
        assert (ref.accept_len == K).any() and ref.trials.max() > 16


@pytest.mark.parametrize("n_trials,weighted", [(3, False), (30, False), (5, True)])
def test_thinning_exhaustion_falls_back_to_the_enumerated_draw(oracle, n_trials, weighted):
    """Keep uniforms just below one: no candidate is kept, every rejected sequence is drawn from the enumerated
    residual with its terminal-group uniform -- which is what pcg_verify's oracle does.  With few supplied trials
    the first eight such sequences of the call are enumerated by a kernel of their own and the others by their own
    blocks; with many, all by their own blocks: both routes must give the oracle's draw."""
    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=5, V=6000, M=1500)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    w = None
    if weighted:
        rng = np.random.default_rng(8)
        raw = rng.random(groups.nnz) + 0.05
        tot = np.zeros(cfg.V)
        np.add.at(tot, groups.group_tok, raw)
        w = (raw / tot[groups.group_tok]).astype(np.float32)
    w64 = None if w is None else w.astype(np.float64)
    tu = W.make_thin_uniforms(cfg, n_trials)
    tu[:, :, 2] = np.float32(1.0 - 2.0 ** -24)
    ref = oracle_thin(oracle, bt, groups, tu, weights=w64)
    plain = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                          groups.tok_degree, bt.uniforms, bt.temperature, weights=w64, threads=0)
    rej = plain.accept_len < cfg.K
    assert rej.sum() > 10 and np.array_equal(ref.tokens[rej], plain.tokens[rej])
    handle = make_handle(groups, weights=w)
    got = run_thin(bt, handle, tu)
    assert_thin_parity(got, ref, max_excused=1 if weighted else 0)
    assert np.all((got[3][rej] & EXHAUSTED) != 0) and np.all(got[4][rej] == n_trials)
    assert np.all((got[3][~rej] & EXHAUSTED) == 0)
    again = run_thin(bt, handle, tu)  # the list order of the shared enumeration may differ from run to run; results may not
    assert all(np.array_equal(x, y) for x, y in zip(got, again))
    # a few trials only: some sequences run out, some do not
    tu2 = W.make_thin_uniforms(cfg, 2)
    ref2 = oracle_thin(oracle, bt, groups, tu2, weights=w64)
    got2 = run_thin(bt, handle, tu2)
    assert_thin_parity(got2, ref2, max_excused=1 if weighted else 0)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_thinning_general_split_weights_and_dtypes(oracle, dtype):
    cfg = W.scaled(W.CONFIGS["C3"], B=32, K=4, V=3000, M=700, dtype=dtype)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    rng = np.random.default_rng(5)
    raw = rng.random(groups.nnz) + 0.05
    tot = np.zeros(cfg.V)
    np.add.at(tot, groups.group_tok, raw)
    w = (raw / tot[groups.group_tok]).astype(np.float32)
    tu = W.make_thin_uniforms(cfg, 32)
    ref = oracle_thin(oracle, bt, groups, tu, weights=w.astype(np.float64))
    assert_thin_parity(run_thin(bt, make_handle(groups, weights=w), tu), ref, max_excused=1)
    ref = oracle_thin(oracle, bt, groups, tu)
    assert_thin_parity(run_thin(bt, make_handle(groups), tu), ref)


def test_thinning_all_accept_masked_logits_and_reproducibility(oracle):
    cfg = W.scaled(W.CONFIGS["C2"], B=8, K=6, V=2048, M=300, emb_dim=16)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    tu = W.make_thin_uniforms(cfg, 24)
    h = make_handle(groups)
    same = W.Batch(bt.target_logits, bt.target_logits[:, :cfg.K].copy(), bt.draft_tokens, bt.uniforms, 1.0, "f32")
    ref = oracle_thin(oracle, same, groups, tu)
    assert np.all(ref.accept_len == cfg.K) and np.all(ref.trials == 1)
    assert_thin_parity(run_thin(same, h, tu), ref)
    # a masked (-inf) stretch of the target row: candidates never come from it
    tl = bt.target_logits.copy()
    tl[:, :, 100:1500] = -np.inf
    masked = W.Batch(tl, bt.draft_logits, bt.draft_tokens, bt.uniforms, 1.0, "f32")
    ref = oracle_thin(oracle, masked, groups, tu)
    got = run_thin(masked, h, tu)
    assert_thin_parity(got, ref)
    for b in range(cfg.B):
        z = got[1][b, got[0][b]]
        assert not (100 <= z < 1500)
    again = run_thin(masked, h, tu)
    assert all(np.array_equal(a, b) for a, b in zip(got, again))


def test_thinning_argument_errors():
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C1"], B=2, K=2)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    tu = W.make_thin_uniforms(cfg, 4)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.PcgError) as ei:
        run_thin(bt, h, tu, workspace=small)
    assert "workspace" in str(ei.value)
    with pytest.raises(binding.PcgError):
        run_thin(bt, h, tu[:, :0])
    got = run_thin(W.Batch(bt.target_logits[:0], bt.draft_logits[:0], bt.draft_tokens[:0], bt.uniforms[:0], 1.0, "f32"),
                   h, tu[:0])
    assert got[0].shape == (0,)


def test_thinning_full_size_bench_configuration_on_sampled_sequences(oracle):
    """C5 as bench.py launches it (B=256, K=16, V=65536, bf16, 32 trials): structure of every sequence, and a
    sample of sequences decision by decision against the oracle."""
    cfg = W.CONFIGS["C5"]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    tu = W.make_thin_uniforms(cfg, 32)
    n, tok, grp, flg, trials = run_thin(bt, make_handle(groups), tu)
    assert np.all((flg & ~EXHAUSTED) == 0) and np.all((n >= 0) & (n <= cfg.K)) and np.all((trials >= 1) & (trials <= 32))
    for b in range(cfg.B):
        assert np.array_equal(tok[b, :n[b]], bt.draft_tokens[b, :n[b]])
        assert np.all(tok[b, n[b] + 1:] == -1) and np.all(grp[b, n[b] + 1:] == -1)
        g = grp[b, n[b]]
        assert tok[b, n[b]] in groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
    sample = list(range(0, cfg.B, 16)) + [int(np.argmax(trials))]
    sub = W.Batch(bt.target_logits[sample], bt.draft_logits[sample], bt.draft_tokens[sample], bt.uniforms[sample],
                  bt.temperature, bt.dtype)
    ref = oracle_thin(oracle, sub, groups, tu[sample])
    assert_thin_parity((n[sample], tok[sample], grp[sample], flg[sample], trials[sample]), ref)
