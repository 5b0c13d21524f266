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


def test_split_vocab_tiles_the_vocabulary():
    assert shard.split_vocab(8, 1) == [(0, 8)]
    for V in (64, 520, 1000, 32000, 128256):
        for world in (1, 2, 3, 8):
            parts = shard.split_vocab(V, world)
            assert len(parts) == world and parts[0][0] == 0 and sum(c for _, c in parts) == V
            for (s0, c0), (s1, _) in zip(parts, parts[1:]):
                assert s1 == s0 + c0 and c0 % 8 == 0 and c0 > 0
            assert parts[-1][1] > 0
    with pytest.raises(ValueError):
        shard.split_vocab(4, 8)
    assert shard.split_vocab(17, 3) == [(0, 8), (8, 8), (16, 1)]
    with pytest.raises(ValueError):
        shard.split_vocab(16, 3)       # two slices of 8 rows leave the third rank nothing


def _vp_worker(rank, world, port, out_path):
    """Each rank scores its slice of the vocabulary with the oracle, writes its slot in the documented
    layout (fp32 logits [rows, k], int32 ids [rows, k], fp32 log-sum-exp [rows]), the slots are
    all-gathered, and the lists folded across ranks must give the unsplit top-k and normaliser."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = small_cfg(d_base=48, d_inner=32, V=200, topk=(3, 2), K=4, B=3, seed=29)
        sw = synth.make_weights(cfg)
        ow = to_oracle_weights(sw)
        ctx, tok = synth.make_draft_inputs(cfg)
        rows, k = cfg.B, cfg.topk[0]
        S = np.stack([oracle.stage_state(ow, 0, oracle.bf16_bits_to_f32(synth.bf16_bits(ctx)[b]), int(tok[b]))
                      for b in range(rows)])
        logits = oracle.stage_logits(ow, 0, S)                     # [rows, V], the unsplit truth
        lo, cnt = shard.split_vocab(cfg.V, world)[rank]
        slot_bytes = -(-(rows * (8 * k + 4)) // 256) * 256
        region = torch.zeros(world, slot_bytes, dtype=torch.uint8)
        val = np.empty((rows, k), np.float32)
        ids = np.empty((rows, k), np.int32)
        lse = np.empty(rows, np.float32)
        for r in range(rows):
            i, v = oracle.topk(logits[r, lo:lo + cnt], k)
            val[r], ids[r], lse[r] = v, i + lo, oracle.logsumexp(logits[r, lo:lo + cnt])
        mine = np.concatenate([val.view(np.uint8).ravel(), ids.view(np.uint8).ravel(), lse.view(np.uint8).ravel()])
        region[rank, :mine.size] = torch.from_numpy(mine)
        shard.all_gather_slots(region, rank, dist)
        ok = True
        for r in range(rows):
            cv, ci, ls = [], [], []
            for g in range(world):
                raw = region[g].numpy()
                cv.append(raw[:rows * k * 4].view(np.float32).reshape(rows, k)[r])
                ci.append(raw[rows * k * 4: rows * k * 8].view(np.int32).reshape(rows, k)[r])
                ls.append(raw[rows * k * 8: rows * k * 8 + rows * 4].view(np.float32)[r])
            cv, ci = np.concatenate(cv), np.concatenate(ci)
            order = np.lexsort((ci, -cv))[:k]                      # value desc, token id asc
            w_i, w_v = oracle.topk(logits[r], k)
            m = max(ls)
            lse_all = m + np.log(sum(np.exp(np.float64(x) - m) for x in ls))
            ok &= np.array_equal(ci[order], w_i) and np.array_equal(cv[order], w_v)
            ok &= abs(lse_all - oracle.logsumexp(logits[r])) < 1e-5
        flags = torch.tensor([1 if ok else 0])
        dist.all_reduce(flags, op=dist.ReduceOp.MIN)
        if rank == 0:
            with open(out_path, "w") as f:
                f.write("ok" if int(flags) == 1 else "mismatch")
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_split_the_vocabulary_and_exchange_lists(tmp_path):
    out = tmp_path / "vp.txt"
    mp.spawn(_vp_worker, args=(2, _free_port(), str(out)), nprocs=2, join=True)
    assert out.read_text() == "ok"
