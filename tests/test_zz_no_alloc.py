"""pcg_verify_static: verification for callers that may not allocate device memory.

Some users of the library run where every byte of device memory was handed out at start-up (a serving process
with its own memory pool, a plug-in inside another application) and cudaMalloc is off limits afterwards; they
cannot provide the workspace pcg_verify asks for.  pcg_verify_static keeps its scratch inside the library image
instead.  This test calls it through the C ABI twice in a row, on different inputs, and checks that it returns
exactly what pcg_verify returns in the same mode -- the second call runs on top of whatever the first left in the
shared scratch --, that both calls agree with the CPU oracle decision by decision, and that calls too large for
the built-in scratch are refused before anything is launched.
This file sorts last so that a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _device_inputs(bt):
    from gpu_util import logits_to_device

    return (logits_to_device(bt.target_logits), logits_to_device(bt.draft_logits),
            torch.from_numpy(bt.draft_tokens).cuda(), torch.from_numpy(bt.uniforms).cuda())


def test_static_scratch_entry_point_matches_pcg_verify_on_two_calls_in_a_row(oracle):
    from gpu_util import make_handle, run_oracle
    from oracle.compare import compare_verify
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=6, V=4000, M=900)
    groups = W.make_groups(cfg)
    handle = make_handle(groups)
    # every tensor the calls need exists before the first call: the entry point itself allocates nothing
    out = (torch.empty(cfg.B, dtype=torch.int32, device="cuda"),
           torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32, device="cuda"),
           torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32, device="cuda"),
           torch.empty(cfg.B, dtype=torch.int32, device="cuda"))
    for call, first_seq in enumerate((0, 500)):
        bt = W.make_batch(cfg, seqs=range(first_seq, first_seq + cfg.B))
        if call == 1:
            bt.draft_logits[::2] = bt.target_logits[::2, :cfg.K]  # long accepts: other positions become terminal
        tl, dl, x, u = _device_inputs(bt)
        want = binding.pcg_verify(tl, dl, x, handle, u, bt.temperature, mode=binding.VERIFY_CLUSTER_TERMINAL)
        for t in out:
            t.fill_(-7)
        binding.pcg_verify_static(tl, dl, x, handle, u, bt.temperature, out)
        torch.cuda.synchronize()
        for got, ref in zip(out, want):
            assert np.array_equal(got.cpu().numpy(), ref.cpu().numpy())  # integer outputs: bit-exact
        # and against the oracle itself, not only against the library's other entry point
        cmp = compare_verify(out[0].cpu().numpy(), out[1].cpu().numpy(), out[2].cpu().numpy(), run_oracle(oracle, bt, groups),
                             band=1e-6)
        assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]
        assert out[0].min().item() >= 0 and out[0].max().item() <= cfg.K
    assert out[0].max().item() == cfg.K  # the second call did reach bonus-token rows


def test_static_scratch_entry_point_refuses_calls_beyond_its_capacity():
    from gpu_util import make_handle
    from paper_2511_13732_b200 import binding

    cfg = W.scaled(W.CONFIGS["C1"], B=2, K=4, V=64, M=8, emb_dim=8)
    handle = make_handle(W.make_groups(cfg))
    B, K = 4096, 32  # 131072 positions: far more bookkeeping than the built-in array holds
    tl = torch.zeros((B, K + 1, cfg.V), dtype=torch.float32, device="cuda")
    dl = torch.zeros((B, K, cfg.V), dtype=torch.float32, device="cuda")
    x = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    u = torch.zeros((B, K + 1, 2), dtype=torch.float32, device="cuda")
    out = (torch.full((B,), -7, dtype=torch.int32, device="cuda"),
           torch.full((B, K + 1), -7, dtype=torch.int32, device="cuda"), None, None)
    with pytest.raises(binding.PcgError) as err:
        binding.pcg_verify_static(tl, dl, x, handle, u, 1.0, out)
    assert err.value.status == 3 and "built-in" in str(err.value)
    torch.cuda.synchronize()
    assert int(out[0].max()) == -7  # refused before any launch: outputs untouched
