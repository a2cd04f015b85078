"""The N > 1 path on CPU: two gloo ranks shard a batch, each verifies its own sequences (here with the oracle
standing in for the GPU call, since only the host logic is under test), and the gathered result equals the
single-process result; the timing reduction takes the max over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_13732_b200 import workloads as W
from paper_2511_13732_b200.sharding import gather_outputs, max_over_ranks, rank_sequences


def test_rank_sequences_partition():
    for B in (0, 1, 7, 16):
        for world in (1, 2, 3, 8):
            strong = [rank_sequences(B, r, world, weak=False) for r in range(world)]
            assert sum(strong, []) == list(range(B))
            assert max(map(len, strong)) - min(map(len, strong)) <= 1
            weak = [rank_sequences(B, r, world, weak=True) for r in range(world)]
            assert sum(weak, []) == list(range(B * world))
    with pytest.raises(ValueError):
        rank_sequences(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import oracle

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = W.scaled(W.CONFIGS["C1"], B=7, K=3, V=256, M=40, emb_dim=8)
        groups = W.make_groups(cfg)
        seqs = rank_sequences(cfg.B, rank, world, weak=False)
        bt = W.make_batch(cfg, seqs=seqs, threads=1)
        res = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                            groups.tok_degree, bt.uniforms, bt.temperature)
        parts = gather_outputs(torch.from_numpy(res.tokens), dist)
        t = max_over_ranks(10.0 + rank, dist)
        if rank == 0:
            q.put((torch.cat(parts).numpy(), t))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_result():
    import oracle

    oracle.build()
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.SimpleQueue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    tokens, t = q.get()
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    cfg = W.scaled(W.CONFIGS["C1"], B=7, K=3, V=256, M=40, emb_dim=8)
    groups = W.make_groups(cfg)
    bt = W.make_batch(cfg)
    ref = oracle.verify(bt.target_logits, bt.draft_logits, bt.draft_tokens, groups.group_ptr, groups.group_tok,
                        groups.tok_degree, bt.uniforms, bt.temperature)
    assert np.array_equal(tokens, ref.tokens)
    assert t == 11.0
