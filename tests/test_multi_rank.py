"""The N > 1 path on CPU: two gloo ranks shard one pairwise matrix by pair-index range and combine it.

The kernel work of a rank is stood in for by the CPU oracle (test infrastructure); what is under test is
the host logic the GPU ranks use: the cost-balanced range partition and the sum all-reduce as gather."""
import os
import socket
import sys

import numpy as np
import pytest
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


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    import roomie_synth as rs
    from paper_2607_16784_b200.shard import combine_shards, partition_pairs

    lib = rs.make_library(1)
    ol = oracle.library_build(lib)
    lo, hi = partition_pairs(lib.offsets, world)[rank]
    Pm, ev = oracle.pair_matrix(ol, n_align=8, start_filter=1, pair_begin=lo, pair_end=hi, num_threads=2)
    mat = torch.from_numpy(Pm.astype(np.float32))
    evals = torch.tensor([ev], dtype=torch.int64)
    combine_shards(mat, evals)
    np.save(os.path.join(out_dir, f"rank{rank}.npy"), mat.numpy())
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{lo} {hi} {int(evals.item())}")
    dist.barrier()
    dist.destroy_process_group()


def test_partition_is_contiguous_disjoint_and_balanced():
    import roomie_synth as rs
    from paper_2607_16784_b200.shard import partition_pairs
    lib = rs.make_library(3, num_profiles=64)
    q = lib.q()
    a, b = np.triu_indices(len(q))
    cost = q[a] + q[b]
    for world in (1, 2, 3, 8):
        parts = partition_pairs(lib.offsets, world)
        assert parts[0][0] == 0 and parts[-1][1] == len(cost)
        assert all(parts[r][1] == parts[r + 1][0] for r in range(world - 1))
        loads = [cost[lo:hi].sum() for lo, hi in parts]
        assert max(loads) - min(loads) <= 2 * cost.max()
    # more ranks than pairs: empty ranges, still a cover
    tiny = partition_pairs([0, 5, 9], 8)
    assert tiny[0][0] == 0 and tiny[-1][1] == 3 and sum(hi - lo for lo, hi in tiny) == 3


def test_two_ranks_shard_and_combine(tmp_path, oracle):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import roomie_synth as rs
    ol = oracle.library_build(rs.make_library(1))
    want, want_ev = oracle.pair_matrix(ol, n_align=8, start_filter=1)
    ranges = []
    for r in range(world):
        got = np.load(tmp_path / f"rank{r}.npy")
        assert np.array_equal(got, want.astype(np.float32))          # every rank holds the full matrix
        lo, hi, ev = (int(x) for x in open(tmp_path / f"rank{r}.txt").read().split())
        ranges.append((lo, hi))
        assert ev == want_ev
    assert ranges[0][1] == ranges[1][0] and ranges[0][0] == 0 and ranges[1][1] == 16 * 17 // 2
    assert 0 < ranges[0][1] < 16 * 17 // 2
