"""world_size-2 `gloo` run on CPU of the multi-rank plumbing: a batch split into per-rank slices of
sequences, drafted and verified independently (by the oracle, standing in for a device) and gathered,
must equal the unsplit batch; step time is the slowest rank's."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2404_19124_b200 import shard, synth
from helpers import small_cfg, to_oracle_weights


def test_split_sequences_covers_the_batch():
    for total in (0, 1, 7, 16, 33):
        for world in (1, 2, 3, 8):
            parts = shard.split_sequences(total, world)
            assert len(parts) == world and sum(c for _, c in parts) == total
            pos = 0
            for s, c in parts:
                assert s == pos and c in (total // world, total // world + 1)
                pos += c
    with pytest.raises(ValueError):
        shard.split_sequences(4, 0)
    assert shard.whole_job_rate(16, 4, 0.5) == 128.0
    assert shard.max_over_ranks(3.5) == 3.5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_path):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = small_cfg(d_base=48, d_inner=32, V=64, topk=(3, 2, 2), K=5, B=5, seed=13)
        sw = synth.make_weights(cfg)
        ow = to_oracle_weights(sw)
        ctx, tok = synth.make_draft_inputs(cfg)
        parts = shard.split_sequences(cfg.B, world)
        s, c = parts[rank]
        ct, lp = oracle.draft(ow, synth.bf16_bits(ctx)[s:s + c], tok.numpy()[s:s + c], cfg.topk, cfg.K)
        cand_all = synth.random_cand_tok(cfg)
        logits = synth.make_base_logits(cfg, cand_all)
        acc, best, nxt = oracle.verify(ct, synth.bf16_bits(logits)[s:s + c], oracle.BF16)
        counts = [p[1] for p in parts]
        g_tok = shard.gather_rows(torch.from_numpy(ct), counts, dist)
        g_acc = shard.gather_rows(torch.from_numpy(np.stack([acc, best, nxt], 1)), counts, dist)
        slow = shard.max_over_ranks(1.0 + rank, dist)      # rank 1 is the slowest
        assert slow == float(world)
        if rank == 0:
            w_tok, _ = oracle.draft(ow, synth.bf16_bits(ctx), tok.numpy(), cfg.topk, cfg.K)
            w = oracle.verify(w_tok, synth.bf16_bits(logits), oracle.BF16)
            ok = np.array_equal(g_tok.numpy(), w_tok) and np.array_equal(g_acc.numpy(), np.stack(w, 1))
            with open(out_path, "w") as f:
                f.write("ok" if ok else "mismatch")
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_the_batch_without_exchanging_data(tmp_path):
    out = tmp_path / "result.txt"
    mp.spawn(_worker, args=(2, _free_port(), str(out)), nprocs=2, join=True)
    assert out.read_text() == "ok"
