"""GPU parity: the CUDA path, called through the C-ABI binding, against the CPU oracle on the same seeded
inputs.  Integer outputs (accept lengths, group ids, tokens) must be identical except where the first differing
decision's uniform lies within 1e-6 of its threshold (counted as excused); P and Q must agree within 1e-5
relative for float32 logits and 1e-3 relative for bf16 logits."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.compare import compare_verify  # noqa: E402

from gpu_util import logits_to_device, make_handle, run_oracle, run_verify  # noqa: E402

BAND = 1e-6
# pcg_verify modes: default (label group per position; per-sequence stage chosen by batch size), dense (P and Q of
# all groups at every position), cluster terminal (one thread-block cluster per sequence), batched terminal
# (transposed residual + sparse product + draw kernels)
MODES = [pytest.param(0, id="default"), pytest.param(1, id="dense"), pytest.param(2, id="cluster"),
         pytest.param(4, id="batched")]


def _assert_parity(got, ref, max_excused=0):
    n, tok, grp, _ = got
    cmp = compare_verify(n, tok, grp, ref, band=BAND)
    assert cmp.hard == 0, f"hard mismatches: {cmp.details[:5]}"
    assert cmp.excused <= max_excused, f"excused mismatches: {cmp.details[:5]}"
    return cmp


# ------------------------------------------------------------------ pcg_group_probs ----
@pytest.mark.parametrize("name,rows", [("C1", 9), ("C2", 40), ("C3", 40), ("C4", 26)])
def test_group_probs_matches_oracle(oracle, name, rows):
    from paper_2511_13732_b200 import binding

    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=max(1, rows // (cfg.K + 1) + 1))
    x = bt.target_logits.reshape(-1, cfg.V)[:rows]
    want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    h = make_handle(groups)
    got = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy().astype(np.float64)
    rtol = 1e-5 if cfg.dtype == "f32" else 1e-3
    np.testing.assert_allclose(got, want, rtol=rtol, atol=1e-37)
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=2e-6)  # no renormalisation is needed (Sec. 2.2)
    # in practice the float32 arithmetic is far inside the bf16 allowance
    assert np.max(np.abs(got - want) / np.maximum(want, 1e-37)) < 1e-5


@pytest.mark.parametrize("name,rows", [("C2", 150), ("C3", 300), ("C4", 64)])
def test_group_probs_batched_route(oracle, name, rows):
    """From 64 rows on pcg_group_probs runs the row-statistics / transposed-operand / sparse-product kernels, a chunk
    of rows at a time (150 and 300 are ragged: not multiples of the 128 rows a warp of the product covers)."""
    from paper_2511_13732_b200 import binding

    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=rows // cfg.K + 1)
    x = np.ascontiguousarray(bt.draft_logits.reshape(-1, cfg.V)[:rows])
    want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    h = make_handle(groups)
    got = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-37)
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=4e-6)
    again = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy()
    assert np.array_equal(again.astype(np.float64), got)  # bit-reproducible
    # the caller-workspace form: same numbers; two calls with separate workspaces on two streams do not disturb each other
    xd = logits_to_device(x)
    ws = [torch.empty(binding.pcg_group_probs_workspace_bytes(cfg.V, groups.M), dtype=torch.uint8, device="cuda") for _ in range(2)]
    outs = [torch.empty((rows, groups.M), dtype=torch.float32, device="cuda") for _ in range(2)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for _ in range(3):
        for k in range(2):
            with torch.cuda.stream(streams[k]):
                binding.pcg_group_probs(xd, h, cfg.temperature, out=outs[k], workspace=ws[k], stream=streams[k])
    torch.cuda.synchronize()
    assert np.array_equal(outs[0].cpu().numpy(), again) and np.array_equal(outs[1].cpu().numpy(), again)
    with pytest.raises(binding.PcgError) as ei:
        binding.pcg_group_probs(xd, h, cfg.temperature, workspace=ws[0][:1024])
    assert ei.value.status == 4
    # with general weights
    rng = np.random.default_rng(3)
    raw = rng.random(groups.nnz) + 0.05
    tot = np.zeros(cfg.V)
    np.add.at(tot, groups.group_tok, raw)
    w = (raw / tot[groups.group_tok]).astype(np.float32)
    want_w = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature,
                                weights=w.astype(np.float64))
    got_w = binding.pcg_group_probs(logits_to_device(x), make_handle(groups, weights=w), cfg.temperature).cpu().numpy()
    np.testing.assert_allclose(got_w, want_w, rtol=1e-5, atol=1e-37)


def test_group_probs_past_one_run_of_row_statistics(oracle):
    """The batched route forms the softmax statistics of sixteen chunks of rows (4096 rows at this size) in one launch;
    4396 rows reach into a second run, whose chunks must pick up their own statistics."""
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], V=1500, M=200, emb_dim=16)
    groups = W.make_groups(cfg)
    rows = 4096 + 300
    bt = W.make_batch(cfg, B=rows // cfg.K + 1)
    x = np.ascontiguousarray(bt.draft_logits.reshape(-1, cfg.V)[:rows])
    want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    h = make_handle(groups)
    got = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(got, want, rtol=1e-3, atol=1e-37)
    assert np.max(np.abs(got - want) / np.maximum(want, 1e-37)) < 1e-5
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=4e-6)


@pytest.mark.parametrize("hint", [1, 2, 4, 8])
def test_group_probs_any_slicing(oracle, hint):
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C4"], V=3000, M=700)  # ragged: V is not a multiple of 64 * slices
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=2)
    x = bt.draft_logits.reshape(-1, cfg.V)
    want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
    h = make_handle(groups, slices_hint=hint)
    assert h.info.slices == hint
    got = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy()
    np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-37)


# ------------------------------------------------------------------------ pcg_verify ----
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4"])
def test_verify_matches_oracle_on_configs(oracle, name, mode):
    cfg = W.CONFIGS[name]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    ref = run_oracle(oracle, bt, groups)
    got = run_verify(bt, make_handle(groups), mode=mode)
    _assert_parity(got, ref)
    assert np.all(got[3] == 0)


@pytest.mark.parametrize("mode", MODES)
def test_verify_c5_shape_small_batch(oracle, mode):
    cfg = W.CONFIGS["C5"]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg, B=12)
    ref = run_oracle(oracle, bt, groups)
    h = make_handle(groups)
    assert h.info.slices == 8
    _assert_parity(run_verify(bt, h, mode=mode), ref)


@pytest.mark.parametrize("mode", MODES)
def test_verify_c5_disjoint_groups_variant(oracle, mode):
    """The disjoint-groups variant of the largest configuration (every token in exactly one of 16384 groups): PCG
    then is standard speculative sampling on the lumped distributions (the oracle is pinned to a textbook
    verifier for exactly this case on the CPU)."""
    cfg = W.CONFIGS["C5d"]
    groups = W.make_groups(cfg)
    assert np.all(groups.tok_degree == 1) and groups.nnz == cfg.V
    bt = W.make_batch(cfg, B=10)
    ref = run_oracle(oracle, bt, groups)
    _assert_parity(run_verify(bt, make_handle(groups), mode=mode), ref)


@pytest.mark.parametrize("mode", [pytest.param(0, id="default"), pytest.param(1, id="dense"), pytest.param(4, id="batched")])
def test_verify_singleton_groups_at_full_vocabulary(oracle, mode):
    """65,536 singleton groups (token-level speculative sampling at the paper's vocabulary size): more groups than
    the 16-bit sweep layout and the draw kernel's shared memory hold, so the handle has no sweep layout, the
    masses are staged in global memory, and the cluster terminal is refused."""
    from paper_2511_13732_b200 import binding

    cfg = W.CONFIGS["C5s"]
    groups = W.make_groups(cfg)
    assert groups.M == 65536
    bt = W.make_batch(cfg, B=6)
    ref = run_oracle(oracle, bt, groups)
    h = make_handle(groups)
    assert h.info.slices == 0
    got = run_verify(bt, h, mode=mode)
    _assert_parity(got, ref)
    assert np.array_equal(got[2][got[2] >= 0], got[1][got[1] >= 0])  # singleton groups: group id = token id
    if mode == 0:
        with pytest.raises(binding.PcgError) as err:
            run_verify(bt, h, mode=2)
        assert err.value.status == 3
        x = bt.target_logits.reshape(-1, cfg.V)[:3]
        want = oracle.softmax(x, cfg.temperature)  # with singleton groups P is the token distribution itself
        P = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy()
        np.testing.assert_allclose(P, want, rtol=1e-5, atol=1e-37)


def test_verify_batch_larger_than_one_chunk_of_the_batched_stage(oracle):
    """At V = 65536 the transposed operand of 256 sequences fills the L2 budget, so 288 sequences run the batched
    per-sequence stage in two chunks (256 + 32)."""
    cfg = W.scaled(W.CONFIGS["C5"], B=288, K=2)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    ref = run_oracle(oracle, bt, groups)
    h = make_handle(groups)
    got = run_verify(bt, h, mode=4)
    _assert_parity(got, ref)
    assert len(set(ref.accept_len[256:].tolist())) > 1  # the second chunk holds different outcomes


def test_verify_batch_spanning_several_sequence_blocks(oracle):
    """The batched per-sequence stage handles 32 sequences per line: 70 sequences = two full blocks and a ragged one,
    with a group count that is not a multiple of the 32 groups a block of the sparse product owns."""
    cfg = W.scaled(W.CONFIGS["C3"], B=70, V=3000, M=1001, K=3)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    bt.draft_logits[::3] = bt.target_logits[::3, :cfg.K]  # every third sequence accepts everything: bonus rows
    ref = run_oracle(oracle, bt, groups)
    assert np.any(ref.accept_len == cfg.K) and np.any(ref.accept_len == 0)
    h = make_handle(groups)
    for mode in (0, 1, 2, 4):
        _assert_parity(run_verify(bt, h, mode=mode), ref)


@pytest.mark.parametrize("B", [130, 300])
def test_verify_wide_sparse_product_forms(oracle, B):
    """From 128 sequences on a lane of the sparse product holds 4 sequences (128-bit loads), from 256 on 8 (256-bit
    loads): ragged batches in both forms, with a group count that is not a multiple of a block's groups, with and
    without general weights, bonus rows included; pcg_group_probs over 300 rows takes the 256-bit form too."""
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], B=B, V=2500, M=611, K=2)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    bt.draft_logits[::5] = bt.target_logits[::5, :cfg.K]
    ref = run_oracle(oracle, bt, groups)
    assert np.any(ref.accept_len == cfg.K) and np.any(ref.accept_len == 0)
    _assert_parity(run_verify(bt, make_handle(groups), mode=4), ref)
    rng = np.random.default_rng(9)
    raw = rng.random(groups.nnz) + 0.05
    tot = np.zeros(cfg.V)
    np.add.at(tot, groups.group_tok, raw)
    w = (raw / tot[groups.group_tok]).astype(np.float32)
    ref_w = run_oracle(oracle, bt, groups, weights=w.astype(np.float64))
    hw = make_handle(groups, weights=w)
    _assert_parity(run_verify(bt, hw, mode=4), ref_w, max_excused=1)
    x = np.ascontiguousarray(bt.target_logits.reshape(-1, cfg.V)[:B])
    want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature,
                              weights=w.astype(np.float64))
    got = binding.pcg_group_probs(logits_to_device(x), hw, cfg.temperature).cpu().numpy()
    np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-37)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("hint", [1, 2, 4, 8])
def test_verify_any_slicing(oracle, hint, mode):
    cfg = W.scaled(W.CONFIGS["C3"], B=24, V=5000, M=1200, K=5)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    ref = run_oracle(oracle, bt, groups)
    _assert_parity(run_verify(bt, make_handle(groups, slices_hint=hint), mode=mode), ref)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("V,dtype", [(1003, "f32"), (1003, "bf16"), (77, "bf16"), (4096 + 8, "bf16"), (5, "f32")])
def test_verify_ragged_and_misaligned_rows(oracle, V, dtype, mode):
    """V not a multiple of the vector width: rows start at unaligned addresses and have scalar heads and tails."""
    cfg = W.scaled(W.CONFIGS["C1"], B=10, K=3, V=V, M=max(2, V // 6), emb_dim=8, dtype=dtype,
                   degree=min(3, max(2, V // 6)))
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    ref = run_oracle(oracle, bt, groups)
    _assert_parity(run_verify(bt, make_handle(groups), mode=mode), ref)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("K", [1, 32, 33, 100])
def test_verify_extreme_k(oracle, K, mode):
    cfg = W.scaled(W.CONFIGS["C1"], B=6, K=K, V=512, M=100, emb_dim=8)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    bt.draft_logits[:] = bt.target_logits[:, :K] + 0.05 * (bt.draft_logits - bt.target_logits[:, :K])  # long accepts
    ref = run_oracle(oracle, bt, groups)
    got = run_verify(bt, make_handle(groups), mode=mode)
    _assert_parity(got, ref)
    if K >= 32:
        assert ref.accept_len.max() > 8
    if K == 100:
        assert ref.accept_len.max() > 32  # first rejection found beyond the first ballot word


@pytest.mark.parametrize("mode", MODES)
def test_verify_with_constant_acceptance_bias(oracle, mode):
    """The lossy relaxation the paper compares against (a constant added to the acceptance ratio, Sec. 3.2)."""
    cfg = W.scaled(W.CONFIGS["C3"], B=48, K=6, V=5000, M=1200)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    plain = run_oracle(oracle, bt, groups)
    biased = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                           groups.tok_degree, bt.uniforms, bt.temperature, accept_bias=float(np.float32(0.3)), threads=0)
    assert biased.accept_len.sum() > plain.accept_len.sum()  # the bias does accept more
    h = make_handle(groups)
    h.set_accept_bias(0.3)
    _assert_parity(run_verify(bt, h, mode=mode), biased)
    h.set_accept_bias(0.0)
    _assert_parity(run_verify(bt, h, mode=mode), plain)


@pytest.mark.parametrize("mode", MODES)
def test_verify_fp16_logits(oracle, mode):
    """IEEE binary16 logits (the third element type) through every mode, plus pcg_group_probs."""
    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=5, V=6000, M=1500, dtype="f16")
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    assert bt.target_logits.dtype == np.float16
    ref = run_oracle(oracle, bt, groups)
    h = make_handle(groups)
    _assert_parity(run_verify(bt, h, mode=mode), ref)
    if mode == 0:
        from paper_2511_13732_b200 import binding

        x = bt.draft_logits.reshape(-1, cfg.V)[:9]
        want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature)
        got = binding.pcg_group_probs(logits_to_device(x), h, cfg.temperature).cpu().numpy()
        np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-37)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_verify_general_split_weights(oracle, dtype, mode):
    """General weights w_{k,t} (non-negative, summing to one over the groups of each token) in place of the equal
    split: the reduction, the label draw and the within-group draw all use them."""
    rng = np.random.default_rng(11)
    cfg = W.scaled(W.CONFIGS["C4"], B=20, K=4, V=3000, M=500, dtype=dtype)
    groups = W.make_groups(cfg)
    raw = rng.random(groups.nnz) + 0.05
    raw[rng.random(groups.nnz) < 0.1] = 0.0  # some memberships carry no mass at all
    tot = np.zeros(cfg.V)
    np.add.at(tot, groups.group_tok, raw)
    dead = tot[groups.group_tok] == 0
    raw[dead] = 1.0
    tot = np.zeros(cfg.V)
    np.add.at(tot, groups.group_tok, raw)
    w = (raw / tot[groups.group_tok]).astype(np.float32)
    bt = W.make_batch(cfg)
    ref = run_oracle(oracle, bt, groups, weights=w.astype(np.float64))
    got = run_verify(bt, make_handle(groups, weights=w), mode=mode)
    _assert_parity(got, ref)
    if mode == 4:
        from paper_2511_13732_b200 import binding

        x = bt.target_logits.reshape(-1, cfg.V)[:7]
        want = oracle.group_probs(x, groups.group_ptr, groups.group_tok, groups.tok_degree, cfg.temperature,
                                  weights=w.astype(np.float64))
        P = binding.pcg_group_probs(logits_to_device(x), make_handle(groups, weights=w), cfg.temperature)
        np.testing.assert_allclose(P.cpu().numpy(), want, rtol=1e-5, atol=1e-37)


def _special_groups(kind, V, rng):
    if kind == "singleton":
        return W.groups_from_lists(V, [[t] for t in range(V)])
    if kind == "one_giant":
        return W.groups_from_lists(V, [list(range(V))])
    if kind == "giant_plus_small":
        return W.groups_from_lists(V, [list(range(V))] + [[t, (t + 1) % V] for t in range(0, V, 7)])
    if kind == "with_empty":
        lists = [[] for _ in range(40)]
        for t in range(V):
            for g in rng.choice(20, size=rng.integers(1, 4), replace=False):
                lists[2 * g].append(t)  # every odd group stays empty
        return W.groups_from_lists(V, lists)
    if kind == "partition":
        a = rng.integers(0, 50, size=V)
        return W.groups_from_lists(V, [list(np.nonzero(a == k)[0]) for k in range(50)])
    raise ValueError(kind)


@pytest.mark.parametrize("kind", ["singleton", "one_giant", "giant_plus_small", "with_empty", "partition"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_verify_degenerate_memberships(oracle, kind, dtype):
    rng = np.random.default_rng(5)
    V, B, K = 2500, 16, 4
    groups = _special_groups(kind, V, rng)
    tl = (2.5 * rng.standard_normal((B, K + 1, V))).astype(np.float32)
    dl = (tl[:, :K] + rng.standard_normal((B, K, V))).astype(np.float32)
    if dtype == "bf16":
        tl, dl = W.f32_to_bf16_bits(tl), W.f32_to_bf16_bits(dl)
    x = rng.integers(0, V, (B, K)).astype(np.int32)
    x[:, 0] = np.argmax(dl[:, 0].astype(np.float32) if dtype == "f32" else W.bf16_bits_to_f32(dl[:, 0]), axis=1)
    u = (rng.integers(0, 1 << 24, (B, K + 1, 2)) * 2.0 ** -24).astype(np.float32)
    bt = W.Batch(tl, dl, x, u, 0.9, dtype)
    ref = run_oracle(oracle, bt, groups)
    for hint, mode in ((0, 4), (0, 1), (0, 2), (4, 1), (4, 2), (4, 0)):
        got = run_verify(bt, make_handle(groups, slices_hint=hint), mode=mode)
        _assert_parity(got, ref)
    if kind == "one_giant":
        assert np.all(ref.accept_len == K)  # a single group is always accepted: P = Q = 1


def test_verify_all_accept_all_reject_and_masked_logits(oracle):
    rng = np.random.default_rng(6)
    cfg = W.scaled(W.CONFIGS["C2"], B=8, K=6, V=2048, M=300, emb_dim=16)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    # identical draft and target: every position accepted, bonus token drawn
    same = W.Batch(bt.target_logits, bt.target_logits[:, :cfg.K].copy(), bt.draft_tokens, bt.uniforms, 1.0, "f32")
    ref = run_oracle(oracle, same, groups)
    assert np.all(ref.accept_len == cfg.K)
    h = make_handle(groups)
    for mode in (0, 1, 2, 4):
        _assert_parity(run_verify(same, h, mode=mode), ref)
    # draft token forced onto a token the target gives no mass (-inf): rejected at position 0
    tl, dl = bt.target_logits.copy(), bt.draft_logits.copy()
    for b in range(cfg.B):
        g_tokens = set()
        for g in range(groups.M):  # mask, in the target, every token that shares a group with the draft token
            toks = groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
            if bt.draft_tokens[b, 0] in toks:
                g_tokens.update(toks.tolist())
        tl[b, 0, list(g_tokens)] = -np.inf
    masked = W.Batch(tl, dl, bt.draft_tokens, bt.uniforms, 1.0, "f32")
    ref = run_oracle(oracle, masked, groups)
    assert np.all(ref.accept_len == 0)
    for mode in (0, 1, 2, 4):
        got = run_verify(masked, h, mode=mode)
        _assert_parity(got, ref)
        assert np.all(got[3] == 0)  # -inf logits are legitimate masks, not an error
    # one dominant logit per row
    tl2 = bt.target_logits.copy()
    tl2[:, :, 17] += 60.0
    dom = W.Batch(tl2, bt.draft_logits, bt.draft_tokens, bt.uniforms, 1.0, "f32")
    ref = run_oracle(oracle, dom, groups)
    for mode in (0, 1, 2, 4):
        _assert_parity(run_verify(dom, h, mode=mode), ref)


def test_verify_is_bit_reproducible_and_flags_bad_tokens(oracle):
    cfg = W.scaled(W.CONFIGS["C3"], B=32)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    first = run_verify(bt, h)
    for _ in range(5):
        again = run_verify(bt, h)
        assert all(np.array_equal(a, b) for a, b in zip(first, again))
    bad = W.Batch(bt.target_logits, bt.draft_logits, bt.draft_tokens.copy(), bt.uniforms, bt.temperature, bt.dtype)
    bad.draft_tokens[3, 0] = cfg.V + 5
    bad.draft_tokens[4, 0] = -1
    got = run_verify(bad, h)
    assert got[3][3] & 1 and got[3][4] & 1 and not np.any(np.delete(got[3], [3, 4]) & 1)
    assert np.all((got[1] >= -1) & (got[1] < cfg.V))


def test_verify_host_entry_point_matches_device_entry_point(oracle):
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], B=16)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    dev = run_verify(bt, h)
    pin = lambda a: torch.from_numpy(a).pin_memory()  # noqa: E731
    tl = torch.from_numpy(bt.target_logits.view(np.int16)).pin_memory()
    dl = torch.from_numpy(bt.draft_logits.view(np.int16)).pin_memory()
    out = (torch.empty(cfg.B, dtype=torch.int32).pin_memory(), torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32).pin_memory(),
           torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32).pin_memory(), torch.empty(cfg.B, dtype=torch.int32).pin_memory())
    need = binding.pcg_verify_host_arena_bytes(cfg.B, cfg.K, cfg.V, groups.M, binding.PCG_BF16)
    arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    binding.pcg_verify_host(tl, dl, pin(bt.draft_tokens), h, pin(bt.uniforms), bt.temperature, arena, out)
    for a, b in zip(dev, out):
        assert np.array_equal(a, b.numpy())
    with pytest.raises(binding.PcgError) as ei:
        binding.pcg_verify_host(tl, dl, pin(bt.draft_tokens), h, pin(bt.uniforms), bt.temperature, arena[:1024], out)
    assert ei.value.status == 4


def test_device_side_argument_errors(oracle):
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C1"], B=2)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    tl, dl = logits_to_device(bt.target_logits), logits_to_device(bt.draft_logits)
    x, u = torch.from_numpy(bt.draft_tokens).cuda(), torch.from_numpy(bt.uniforms).cuda()
    with pytest.raises(binding.PcgError) as ei:
        binding.pcg_verify(tl, dl, x, h, u, 0.0)
    assert ei.value.status == 1
    with pytest.raises(binding.PcgError) as ei:
        binding.pcg_verify(tl, dl, x, h, u, 1.0, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert ei.value.status == 4
    # B = 0 and rows = 0 are no-ops
    binding.pcg_verify(tl[:0], dl[:0], x[:0], h, u[:0], 1.0)
    assert binding.pcg_group_probs(tl.reshape(-1, cfg.V)[:0], h).shape == (0, groups.M)


@pytest.mark.parametrize("mode", [pytest.param(0, id="default"), pytest.param(1, id="dense"),
                                  pytest.param(2, id="cluster")])
def test_full_size_bench_configuration_on_sampled_sequences(oracle, mode):
    """C5 exactly as bench.py launches it (B=256, K=16, V=65536, bf16): every sequence is checked for structure,
    and a sample of sequences is checked decision by decision against the oracle."""
    cfg = W.CONFIGS["C5"]
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    h = make_handle(groups)
    n, tok, grp, flg = run_verify(bt, h, mode=mode)
    assert np.all(flg == 0) and np.all((n >= 0) & (n <= cfg.K))
    for b in range(cfg.B):
        assert np.array_equal(tok[b, :n[b]], bt.draft_tokens[b, :n[b]])
        assert np.all(tok[b, n[b] + 1:] == -1) and np.all(grp[b, n[b] + 1:] == -1)
        for i in range(n[b] + 1):
            g = grp[b, i]
            assert tok[b, i] in groups.group_tok[groups.group_ptr[g]:groups.group_ptr[g + 1]]
    sample = list(range(0, cfg.B, 16)) + [int(np.argmax(n))]
    sub = W.Batch(bt.target_logits[sample], bt.draft_logits[sample], bt.draft_tokens[sample], bt.uniforms[sample],
                  bt.temperature, bt.dtype)
    ref = run_oracle(oracle, sub, groups)
    _assert_parity((n[sample], tok[sample], grp[sample], flg[sample]), ref)

@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rows_that_rise_far_above_their_start(oracle, dtype, mode):
    """The streaming kernel sums a thread's vectors against the reference its FIRST vector set and checks the
    running sum once per row; a row whose logits climb by hundreds of nats makes that sum overflow (or exceed the
    limit) in most threads, which then form their sums again with the reference raised as they go.  Rising,
    falling and saw-tooth rows, against the oracle."""
    cfg = W.scaled(W.CONFIGS["C3"], B=9, K=3, V=20000, M=3000, emb_dim=16, dtype=dtype)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    rng = np.random.default_rng(77)
    t = np.arange(cfg.V, dtype=np.float64) / cfg.V
    shapes = [-300.0 + 600.0 * t, 300.0 - 600.0 * t, 250.0 * np.abs(((7.0 * t) % 2.0) - 1.0) - 125.0]

    def reshape(a, scale):
        rows = a.shape[0] * a.shape[1]
        out = np.empty((rows, cfg.V), np.float64)
        for r in range(rows):
            out[r] = scale * shapes[r % 3] + 2.0 * rng.standard_normal(cfg.V)
        out = out.reshape(a.shape).astype(np.float32)
        return W.f32_to_bf16_bits(out) if dtype == "bf16" else out

    tl, dl = reshape(bt.target_logits, 1.0), reshape(bt.draft_logits, 0.97)
    # drafted tokens among the 200 likeliest of their draft row (a token of vanishing mass has no float32 ratio to test)
    dl32 = W.bf16_bits_to_f32(dl) if dtype == "bf16" else dl
    x = np.empty_like(bt.draft_tokens)
    for b in range(cfg.B):
        for i in range(cfg.K):
            x[b, i] = rng.choice(np.argpartition(-dl32[b, i], 200)[:200])
    hard = W.Batch(tl, dl, x, bt.uniforms, bt.temperature, dtype)
    ref = run_oracle(oracle, hard, groups)
    got = run_verify(hard, make_handle(groups), mode=mode)
    _assert_parity(got, ref, max_excused=1)
    assert np.all(got[3] == 0)
