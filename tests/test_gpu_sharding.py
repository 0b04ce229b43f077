"""The data-parallel chain on real kernels: shard_indices -> CUDA forward per shard -> gather_embeddings,
run by two ranks (gloo for the gather, both using cuda:0; the ranks' kernels never wait on each other)
and compared bitwise with the unsharded forward."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402

from synth.inputs import CONFIGS, EncoderConfig, make_inputs  # noqa: E402

pytestmark = pytest.mark.gpu

CFG = CONFIGS["c2"]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _forward(rlx, cfg, ids, mask, params, layers):
    sub = EncoderConfig(**{**cfg.__dict__, "batch": ids.shape[0]})
    enc = rlx.Encoder.from_config(sub, max_batch=sub.batch, max_seq=sub.seq)
    w = rlx.upload_weights(params, layers)
    ws = enc.alloc_workspace(sub.batch, sub.seq)
    out = torch.empty((sub.batch, sub.hidden), dtype=torch.float32, device="cuda")
    enc.forward(torch.from_numpy(ids).cuda(), torch.from_numpy(mask).cuda(), w, out, ws)
    torch.cuda.synchronize()
    assert enc.last_device_status(ws) == 0
    enc.close()
    return out.cpu()


def _worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import paper_2609_37916_b200 as rlx
        from paper_2609_37916_b200.sharding import gather_embeddings, shard_indices
        torch.cuda.set_device(0)
        inp = make_inputs(CFG)
        shards = shard_indices(inp.lengths, world)
        mine = shards[rank]
        local = _forward(rlx, CFG, np.ascontiguousarray(inp.ids[mine]), np.ascontiguousarray(inp.mask[mine]), inp.params, inp.layers)
        full = gather_embeddings(local, shards, CFG.batch)
        if rank == 0:
            ret["full"] = full.numpy()
    finally:
        dist.destroy_process_group()


def test_two_rank_sharded_cuda_forward_equals_unsharded_bitwise():
    import paper_2609_37916_b200 as rlx
    from paper_2609_37916_b200.build import build
    build()
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    inp = make_inputs(CFG)
    whole = _forward(rlx, CFG, inp.ids, inp.mask, inp.params, inp.layers).numpy()
    # sequences are independent and every reduction has a fixed order: sharding changes nothing, bit for bit
    assert np.array_equal(ret["full"], whole)
