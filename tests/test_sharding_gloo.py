"""Multi-rank host logic on CPU: two `gloo` ranks shard the rows, run the oracle on their own
rows and combine -- the result must equal the unsharded oracle."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_22347_b200 import inputs, sharding


def test_row_shard_covers_every_row_once():
    for T in (0, 1, 5, 16, 16384, 16385):
        for world in (1, 2, 3, 8):
            spans = [sharding.row_shard(T, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import perq_oracle
    T, d, b = 37, 256, 32
    bits, _ = inputs.swiglu_outliers(T, d, 4, 30.0, seed=910)
    perm = inputs.random_perm(d, 911)
    lo, hi = sharding.row_shard(T, rank, world)
    # the statistic on this rank's rows, then the exchange
    cas, blm, tmx = perq_oracle.block_l1_stats(bits[lo:hi], perm, b)
    chan, block = torch.from_numpy(cas.copy()), torch.from_numpy(blm.copy())
    total = sharding.allreduce_block_l1_stats(chan, block, hi - lo)
    # rotate+quantize of this rank's rows: no exchange, outputs are row ranges
    ora = perq_oracle.rotate_quantize(bits[lo:hi], perm, b, perq_oracle.FMT_MXFP4, 32)
    slowest = sharding.max_over_ranks(1.0 + rank)
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), chan=chan.numpy(), block=block.numpy(), tmx=tmx,
             codes=ora["codes"], scales=ora["scales"], total=total, slowest=slowest, lo=lo, hi=hi)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_result(tmp_path, oracle):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    T, d, b = 37, 256, 32
    bits, _ = inputs.swiglu_outliers(T, d, 4, 30.0, seed=910)
    perm = inputs.random_perm(d, 911)
    cas, blm, tmx = oracle.block_l1_stats(bits, perm, b)
    full = oracle.rotate_quantize(bits, perm, b, oracle.FMT_MXFP4, 32)
    parts = [np.load(os.path.join(str(tmp_path), "rank%d.npz" % r)) for r in range(world)]
    for p in parts:
        assert int(p["total"]) == T and float(p["slowest"]) == 2.0
        assert np.allclose(p["chan"], cas, rtol=1e-12) and np.allclose(p["block"], blm, rtol=1e-12)
    assert np.array_equal(np.concatenate([p["tmx"] for p in parts]), tmx)
    assert np.array_equal(np.concatenate([p["codes"] for p in parts]), full["codes"])
    assert np.array_equal(np.concatenate([p["scales"] for p in parts]), full["scales"])
