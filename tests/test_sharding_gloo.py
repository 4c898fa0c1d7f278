"""world_size-2 gloo test of the multi-GPU host logic: row partition, per-rank oracle
selection equals the unsharded selection, max-over-ranks timing reduction."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, tmpdir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import topk_definition as D
    from paper_2609_08450_b200 import sharding, workloads as W
    batch = W.config1(seed=99, num_rows=12, max_len=3000, K=64)
    scores, starts, lengths = batch.host()
    parts = sharding.partition_rows(lengths, world)
    b, e = parts[rank]
    idx, _ = D.topk_rows(scores, starts[b:e], lengths[b:e], 64)
    np.save(os.path.join(tmpdir, f"idx{rank}.npy"), idx)
    t = sharding.max_over_ranks(10.0 + rank)
    s = sharding.sum_over_ranks(float(np.clip(lengths[b:e], 0, None).sum()))
    assert t == 10.0 + world - 1
    assert s == float(np.clip(lengths, 0, None).sum())
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_row_sharding(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import topk_definition as D
    from paper_2609_08450_b200 import sharding, workloads as W
    batch = W.config1(seed=99, num_rows=12, max_len=3000, K=64)
    scores, starts, lengths = batch.host()
    whole, _ = D.topk_rows(scores, starts, lengths, 64)
    got = np.concatenate([np.load(tmp_path / f"idx{r}.npy") for r in range(world)])
    assert np.array_equal(got, whole)
    parts = sharding.partition_rows(lengths, world)
    assert parts[0][0] == 0 and parts[-1][1] == len(lengths) and parts[0][1] == parts[1][0]
    loads = [int(np.clip(lengths[b:e], 0, None).sum()) for b, e in parts]
    assert max(loads) - min(loads) <= 2 * int(lengths.max())


def test_partition_edge_cases():
    sys.path.insert(0, ROOT)
    from paper_2609_08450_b200 import sharding
    assert sharding.partition_rows([], 2) == [(0, 0), (0, 0)]
    assert sharding.partition_rows([5], 4)[-1][1] == 1
    parts = sharding.partition_rows([1, 1, 1, 1, 100], 2)
    assert parts[0][1] == parts[1][0] and parts[1][1] == 5
    assert sharding.partition_rows([-5, 0, 3], 1) == [(0, 3)]
