"""Tensor-parallel sharding on CPU (gloo, world_size 2 and 4): the parameter shards of
tensor_parallel.shard_weights_tp, run through the oracle's stage functions with an all-reduce after each
row-parallel product, reproduce the single-rank oracle.  This pins the shard layout (which rows and
columns a rank holds, q | k | v order, biases counted once) without a GPU."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37916_b200.tensor_parallel import check_tp, shard_layer_tp, shard_weights_tp
from synth.inputs import EncoderConfig, make_inputs

CFG = EncoderConfig("tp_small", 2, 256, 8, 512, 5, 24, 2, 24, 3, vocab=131, max_pos=32)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_check_tp_accepts_whole_heads_and_64_wide_blocks_only():
    check_tp(12, 384, 1536, 2)
    check_tp(12, 384, 1536, 3)
    check_tp(12, 384, 1536, 6)
    for bad in (4, 5, 12):      # 96-wide shards, heads not divisible, 32-wide shards
        with pytest.raises(ValueError):
            check_tp(12, 384, 1536, bad)


def test_shards_tile_the_full_matrices():
    inp = make_inputs(CFG)
    lw = inp.layers[0]
    H, F, world = CFG.hidden, CFG.ffn, 4
    parts = [shard_layer_tp(lw, r, world, CFG.num_heads) for r in range(world)]
    # row-parallel matrices: the column blocks side by side give the matrix back
    assert np.array_equal(np.concatenate([p["wo"] for p in parts], axis=1), lw["wo"])
    assert np.array_equal(np.concatenate([p["w2"] for p in parts], axis=1), lw["w2"])
    assert np.array_equal(np.concatenate([p["w1"] for p in parts], axis=0), lw["w1"])
    # column-parallel qkv: rank r's block is [q rows | k rows | v rows] of its heads
    Hl = H // world
    for r, p in enumerate(parts):
        for part in range(3):
            assert np.array_equal(p["wqkv"][part * Hl:(part + 1) * Hl], lw["wqkv"][part * H + r * Hl: part * H + (r + 1) * Hl])
            assert np.array_equal(p["bqkv"][part * Hl:(part + 1) * Hl], lw["bqkv"][part * H + r * Hl: part * H + (r + 1) * Hl])
    # the row-parallel biases are counted once
    assert np.array_equal(sum(p["bo"] for p in parts), lw["bo"]) and np.array_equal(sum(p["b2"] for p in parts), lw["b2"])
    assert all(np.array_equal(p["ln1_g"], lw["ln1_g"]) for p in parts)


def _tp_forward_with_oracle(oracle, rank, world, x_emb, mask, shard_layers, cfg):
    def allreduce(a):
        t = torch.from_numpy(a)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return t.numpy()

    x = x_emb
    h_loc = cfg.num_heads // world
    for lw in shard_layers:
        qkv = oracle.linear(x, lw["wqkv"], lw["bqkv"])
        ctx = oracle.attention(qkv, mask, h_loc)
        y = oracle.linear(ctx, lw["wo"], lw["bo"])
        if rank == 0:
            y = y + x
        x1 = oracle.layernorm(allreduce(y), lw["ln1_g"], lw["ln1_b"], cfg.ln_eps)
        g = oracle.gelu(oracle.linear(x1, lw["w1"], lw["b1"]))
        y = oracle.linear(g, lw["w2"], lw["b2"])
        if rank == 0:
            y = y + x1
        x = oracle.layernorm(allreduce(y), lw["ln2_g"], lw["ln2_b"], cfg.ln_eps)
    return oracle.pool_l2(x, mask)


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import oracle
        inp = make_inputs(CFG)
        _, dumps = oracle.encoder_forward(CFG, inp.ids, inp.mask, inp.params, inp.layers, compute_all_rows=True, dumps=True)
        shard = shard_weights_tp(inp.layers, rank, world, CFG.num_heads)
        out = _tp_forward_with_oracle(oracle, rank, world, dumps["x_emb"], inp.mask, shard, CFG)
        ret[rank] = out
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_tensor_parallel_ranks_reproduce_the_single_rank_oracle(world):
    from oracle import oracle
    oracle.build()
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    inp = make_inputs(CFG)
    ref = oracle.encoder_forward(CFG, inp.ids, inp.mask, inp.params, inp.layers)
    for r in range(world):
        assert np.abs(ret[r] - ref).max() <= 1e-12      # fp64: only the order of the partial sums differs
    assert np.array_equal(ret[0], ret[1])                # every rank ends with the same embeddings
