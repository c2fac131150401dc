"""The N > 1 layout on CPU: two gloo ranks shard the sequences, compress their shards with the
oracle (standing in for the per-rank library context), and the gathered result equals the
single-process one -- the path needs no data collective, only the walk seed offset."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import OracleParams, OracleStream
from paper_2502_07861_b200 import shard, synth

N_SEQS, N, D, T_BLOCK, LEVELS, BASE_SEED = 5, 96, 8, 16, 2, 11


def _compress_sequence(global_seq, local_seq, ctx_seed):
    """What a rank's context does for its local sequence `local_seq` (coin key = ctx_seed + local)."""
    K, V = synth.stream_kv("outlier2", 77, global_seq, 0, 0, N, D, "fp32")
    s = OracleStream(OracleParams(d=D, t=T_BLOCK, T=LEVELS, max_tokens=N, seed=ctx_seed + local_seq, c_override=0.5))
    s.append(K, V)
    s.compress()
    return s.view()[3].astype(np.int64)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = shard.shard_range(N_SEQS, world, rank)
    seed = shard.walk_seed(BASE_SEED, mine.start)
    kept = [_compress_sequence(g, g - mine.start, seed) for g in mine]
    # output gather (not part of the path): ranks hold different numbers of sequences
    gathered = [None] * world
    dist.all_gather_object(gathered, (list(mine), [k.tolist() for k in kept]))
    t = shard.max_over_ranks(10.0 + rank)
    if rank == 0:
        np.save(os.path.join(out_dir, "t.npy"), np.array([t]))
        torch.save(gathered, os.path.join(out_dir, "gathered.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_sequences_without_exchange(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    gathered = torch.load(os.path.join(tmp_path, "gathered.pt"), weights_only=False)
    assert float(np.load(os.path.join(tmp_path, "t.npy"))[0]) == 11.0          # max over ranks
    owned = [g for part in gathered for g in part[0]]
    assert owned == list(range(N_SEQS))                                       # disjoint, complete, ordered
    single = [_compress_sequence(g, g, BASE_SEED) for g in range(N_SEQS)]
    multi = [np.array(k) for part in gathered for k in part[1]]
    for a, b in zip(single, multi):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("n,world", [(0, 1), (1, 4), (5, 2), (8, 8), (13, 4), (7, 3)])
def test_shard_range_partitions(n, world):
    parts = [shard.shard_range(n, world, r) for r in range(world)]
    assert [i for p in parts for i in p] == list(range(n))
    assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
    for r, p in enumerate(parts):
        for i in p:
            assert shard.owner_of(i, n, world) == r
    with pytest.raises(ValueError):
        shard.shard_range(n, world, world)
