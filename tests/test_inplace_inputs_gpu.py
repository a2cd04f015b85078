"""A decoding loop refills the SAME device buffers before every call.  Several kernels of a call read inputs (uniforms,
draft tokens, trial uniforms) and results of earlier kernels ahead of their programmatic wait for the kernel in
front; whatever a call reads must be what the buffers hold when it is enqueued, never a copy of an earlier call's
contents.  Back-to-back calls on refilled buffers, no synchronisation in between, each checked against the oracle."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.compare import compare_verify  # noqa: E402

from gpu_util import logits_to_device, make_handle, run_oracle  # noqa: E402
from test_thinning_gpu import assert_thin_parity, oracle_thin  # noqa: E402

ROUNDS = 6


def _batches(cfg, per_round):
    """Disjoint runs of sequences of one configuration: round r holds sequences r*per_round ..."""
    return [W.make_batch(cfg, seqs=range(r * per_round, (r + 1) * per_round)) for r in range(ROUNDS)]


@pytest.mark.parametrize("mode", [pytest.param(0, id="default"), pytest.param(4, id="batched"), pytest.param(2, id="cluster")])
def test_verify_on_refilled_buffers(oracle, mode):
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=6, V=5000, M=900, emb_dim=16)
    groups = W.make_groups(cfg)
    h = make_handle(groups)
    rounds = _batches(cfg, cfg.B)
    dev = [logits_to_device(rounds[0].target_logits).clone(), logits_to_device(rounds[0].draft_logits).clone(),
           torch.from_numpy(rounds[0].draft_tokens).cuda(), torch.from_numpy(rounds[0].uniforms).cuda()]
    staged = [(logits_to_device(bt.target_logits), logits_to_device(bt.draft_logits), torch.from_numpy(bt.draft_tokens).cuda(),
               torch.from_numpy(bt.uniforms).cuda()) for bt in rounds]
    ws = torch.empty(binding.pcg_verify_workspace_bytes(cfg.B, cfg.K, cfg.V, groups.M, binding.PCG_BF16, mode), dtype=torch.uint8,
                     device="cuda")
    torch.cuda.synchronize()
    outs = []
    for r in range(ROUNDS):  # refill and call, all on one stream, nothing waited for
        for d, s in zip(dev, staged[r]):
            d.copy_(s)
        out = binding.pcg_verify(dev[0], dev[1], dev[2], h, dev[3], cfg.temperature, mode=mode, workspace=ws)
        outs.append(tuple(o.clone() for o in out))
    torch.cuda.synchronize()
    for r in range(ROUNDS):
        n, tok, grp, flg = (o.cpu().numpy() for o in outs[r])
        cmp = compare_verify(n, tok, grp, run_oracle(oracle, rounds[r], groups))
        assert cmp.hard == 0 and cmp.excused == 0, (r, cmp.details[:3])
        assert np.all(flg == 0)


def test_thinning_on_refilled_buffers(oracle):
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=6, V=5000, M=900, emb_dim=16)
    groups = W.make_groups(cfg)
    h = make_handle(groups)
    rounds = _batches(cfg, cfg.B)
    tus = [W.make_thin_uniforms(cfg, 12, seqs=range(r * cfg.B, (r + 1) * cfg.B)) for r in range(ROUNDS)]
    dev = [logits_to_device(rounds[0].target_logits).clone(), logits_to_device(rounds[0].draft_logits).clone(),
           torch.from_numpy(rounds[0].draft_tokens).cuda(), torch.from_numpy(rounds[0].uniforms).cuda(),
           torch.from_numpy(tus[0]).cuda()]
    staged = [(logits_to_device(bt.target_logits), logits_to_device(bt.draft_logits), torch.from_numpy(bt.draft_tokens).cuda(),
               torch.from_numpy(bt.uniforms).cuda(), torch.from_numpy(tu).cuda()) for bt, tu in zip(rounds, tus)]
    torch.cuda.synchronize()
    outs = []
    for r in range(ROUNDS):
        for d, s in zip(dev, staged[r]):
            d.copy_(s)
        out = binding.pcg_verify_thinning(dev[0], dev[1], dev[2], h, dev[3], dev[4], cfg.temperature)
        outs.append(tuple(o.clone() for o in out))
    torch.cuda.synchronize()
    for r in range(ROUNDS):
        got = tuple(o.cpu().numpy() for o in outs[r])
        assert_thin_parity(got, oracle_thin(oracle, rounds[r], groups, tus[r]), max_excused=1)
