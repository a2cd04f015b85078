"""pcg_verify only enqueues kernels on the caller's stream (no allocation, no synchronisation), so a call can be
captured into a CUDA graph and replayed on new inputs written into the same buffers."""
import numpy as np
import pytest

from paper_2511_13732_b200 import workloads as W

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [pytest.param(2, id="cluster"), pytest.param(4, id="batched")])
def test_captured_call_replays_on_new_inputs(oracle, mode):
    from oracle.compare import compare_verify
    from paper_2511_13732_b200 import binding

    from gpu_util import logits_to_device, make_handle, run_oracle

    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=4, V=4096, M=1000)
    groups = W.make_groups(cfg)
    handle = make_handle(groups)
    first, second = W.make_batch(cfg, seqs=range(0, 40)), W.make_batch(cfg, seqs=range(100, 140))
    tl, dl = logits_to_device(first.target_logits), logits_to_device(first.draft_logits)
    x, u = torch.from_numpy(first.draft_tokens).cuda(), torch.from_numpy(first.uniforms).cuda()
    ws = torch.empty(binding.pcg_verify_workspace_bytes(cfg.B, cfg.K, cfg.V, groups.M, binding.PCG_BF16, mode),
                     dtype=torch.uint8, device="cuda")
    out = (torch.empty(cfg.B, dtype=torch.int32, device="cuda"), torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32, device="cuda"),
           torch.empty((cfg.B, cfg.K + 1), dtype=torch.int32, device="cuda"), torch.empty(cfg.B, dtype=torch.int32, device="cuda"))
    binding.pcg_verify(tl, dl, x, handle, u, cfg.temperature, workspace=ws, out=out, mode=mode)  # warm-up, sets attributes
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.pcg_verify(tl, dl, x, handle, u, cfg.temperature, workspace=ws, out=out, mode=mode)
    for batch in (second, first):
        tl.copy_(logits_to_device(batch.target_logits))
        dl.copy_(logits_to_device(batch.draft_logits))
        x.copy_(torch.from_numpy(batch.draft_tokens))
        u.copy_(torch.from_numpy(batch.uniforms))
        for t in out:
            t.fill_(-9)
        graph.replay()
        torch.cuda.synchronize()
        ref = run_oracle(oracle, batch, groups)
        cmp = compare_verify(out[0].cpu().numpy(), out[1].cpu().numpy(), out[2].cpu().numpy(), ref)
        assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]


def test_captured_thinning_call_replays_on_new_inputs(oracle):
    from oracle.compare import compare_verify
    from paper_2511_13732_b200 import binding

    from gpu_util import library_candidate_order, logits_to_device, make_handle

    cfg = W.scaled(W.CONFIGS["C3"], B=40, K=4, V=4096, M=1000)
    groups = W.make_groups(cfg)
    handle = make_handle(groups)
    tl = torch.empty((cfg.B, cfg.K + 1, cfg.V), dtype=torch.bfloat16, device="cuda")
    dl = torch.empty((cfg.B, cfg.K, cfg.V), dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((cfg.B, cfg.K), dtype=torch.int32, device="cuda")
    u = torch.zeros((cfg.B, cfg.K + 1, 2), dtype=torch.float32, device="cuda")
    tu = torch.zeros((cfg.B, 24, 3), dtype=torch.float32, device="cuda")
    ws = torch.empty(binding.pcg_verify_thinning_workspace_bytes(cfg.B, cfg.K, cfg.V, groups.M, binding.PCG_BF16),
                     dtype=torch.uint8, device="cuda")
    out = None
    graph = None
    for seqs in (range(0, 40), range(100, 140), range(0, 40)):
        batch, thin = W.make_batch(cfg, seqs=seqs), W.make_thin_uniforms(cfg, 24, seqs=seqs)
        tl.copy_(logits_to_device(batch.target_logits))
        dl.copy_(logits_to_device(batch.draft_logits))
        x.copy_(torch.from_numpy(batch.draft_tokens))
        u.copy_(torch.from_numpy(batch.uniforms))
        tu.copy_(torch.from_numpy(thin))
        if graph is None:  # first batch: a plain call (sets the kernel attributes), then the capture
            out = binding.pcg_verify_thinning(tl, dl, x, handle, u, tu, cfg.temperature, workspace=ws)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                binding.pcg_verify_thinning(tl, dl, x, handle, u, tu, cfg.temperature, workspace=ws, out=out)
        for t in out:
            t.fill_(-9)
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.verify(batch.target_logits, batch.draft_logits, batch.draft_tokens, groups.group_ptr,
                            groups.group_tok, groups.tok_degree, batch.uniforms, batch.temperature, threads=0,
                            thin_uniforms=thin, cand_order=library_candidate_order(groups.V, batch.target_logits))
        cmp = compare_verify(out[0].cpu().numpy(), out[1].cpu().numpy(), out[2].cpu().numpy(), ref)
        assert cmp.hard == 0 and cmp.excused == 0, cmp.details[:3]
        assert np.array_equal(out[4].cpu().numpy(), ref.trials)
