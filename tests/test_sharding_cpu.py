"""N > 1 host logic on CPU: two gloo ranks shard a token batch, run a row-wise function on
their slices and agree on a max-reduced timing.  No GPU, no collective on the data path."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_token_shard_tiles_the_batch():
    from paper_2604_07853_b200.sharding import token_shard
    for m in (0, 1, 7, 64, 1000, 32768):
        for w in (1, 2, 3, 8):
            spans = [token_shard(m, w, r) for r in range(w)]
            assert spans[0][0] == 0 and spans[-1][1] == m
            assert all(spans[i][1] == spans[i + 1][0] for i in range(w - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        token_shard(10, 2, 2)


def _worker(rank: int, world: int, port: int, tmp: str):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2604_07853_b200 import inputs
    from paper_2604_07853_b200.sharding import max_over_ranks, token_shard
    import oracle
    # every rank draws the same batch from the seed, takes its slice and runs a row-wise
    # stage of the path on it (the oracle's activation quantizer stands in for the GPU call)
    x = inputs.act_bf16(np.random.default_rng(0), 37, 256)
    b, e = token_shard(37, world, rank)
    codes, scales = oracle.quantize_act(x[b:e])
    np.save(os.path.join(tmp, f"codes{rank}.npy"), codes)
    np.save(os.path.join(tmp, f"scales{rank}.npy"), scales)
    got = max_over_ranks(1.0 + rank)
    assert got == float(world)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharded_run_equals_unsharded(tmp_path):
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2604_07853_b200 import inputs
    x = inputs.act_bf16(np.random.default_rng(0), 37, 256)
    codes, scales = oracle.quantize_act(x)
    cat_c = np.concatenate([np.load(tmp_path / f"codes{r}.npy") for r in range(2)])
    cat_s = np.concatenate([np.load(tmp_path / f"scales{r}.npy") for r in range(2)])
    assert np.array_equal(cat_c, codes) and np.array_equal(cat_s, scales)
