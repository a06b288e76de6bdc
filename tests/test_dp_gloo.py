"""The N > 1 path on CPU: two gloo ranks shard a global batch, run their slices (through the
oracle here -- no GPU), and agree on the max-over-ranks time; together they cover the batch."""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, str(ROOT))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2101_01321_b200 import dp, synth
    B, L, H, heads, F = 5, 16, 128, 2, 256           # 5 sequences over 2 ranks: 3 + 2
    x, params = synth.make_model(0, B, layers=1, H=H, heads=heads, F=F, L=L)
    first, last = dp.shard_range(B, world, rank)
    mine = x[first * L:last * L]
    out = oracle.encoder_layer(params[0], mine, last - first, L).out
    np.save(Path(out_dir) / f"out_{rank}.npy", out)
    ms = dp.max_over_ranks([10.0 + rank, 5.0 - rank])
    assert ms == [10.0 + world - 1, 5.0]
    dist.barrier()
    dist.destroy_process_group()


def test_shard_range_covers_the_batch_without_overlap():
    from paper_2101_01321_b200 import dp
    for B in (0, 1, 5, 128, 1000):
        for world in (1, 2, 3, 8):
            spans = [dp.shard_range(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        dp.shard_range(4, 2, 2)


def test_two_gloo_ranks_reproduce_the_single_process_result(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    sys.path.insert(0, str(ROOT))
    import oracle
    from paper_2101_01321_b200 import synth
    x, params = synth.make_model(0, 5, layers=1, H=128, heads=2, F=256, L=16)
    whole = oracle.encoder_layer(params[0], x, 5, 16).out
    parts = np.concatenate([np.load(tmp_path / f"out_{r}.npy") for r in range(2)])
    assert np.array_equal(parts, whole)        # sequences are independent: sharding changes nothing
