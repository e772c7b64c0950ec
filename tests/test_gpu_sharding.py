"""The sharded pairwise matrix on the GPU: pair-index ranges computed one after the other (as the ranks of a
multi-GPU run would compute them side by side) add up to the single-call matrix bit for bit."""
import os
import socket
import sys

import numpy as np
import pytest

import roomie_synth as rs

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("gpu-marked test run without a CUDA device")
    import paper_2607_16784_b200 as rm
    return torch, rm


@pytest.mark.parametrize("kw", [dict(mode=0, n_align=1, start_filter=0), dict(mode=0, n_align=8, start_filter=1),
                                dict(mode=2, n_align=4, start_filter=1)])
def test_four_rank_ranges_sum_to_the_single_call(kw):
    """World size 4 emulated on one GPU: every rank's range goes into a zeroed matrix of its own; the sum of
    the four (what the all-reduce computes) equals the matrix of one call over all pairs, and so do the counts."""
    torch, rm = _gpu()
    from paper_2607_16784_b200.shard import partition_pairs
    lib = rs.make_library(3, num_profiles=48)
    gl = rm.library_build(lib.grid_blocks, lib.block_threads, lib.regs_per_thread, lib.smem_per_block,
                          lib.dur_us, lib.gap_us, lib.offsets, lib.spec)
    full, ev_full = rm.pair_matrix(gl, **kw)
    parts = partition_pairs(lib.offsets, 4)
    assert parts[0][0] == 0 and parts[-1][1] == 48 * 49 // 2 and all(hi > lo for lo, hi in parts)
    total = torch.zeros_like(full)
    evals = 0
    touched = torch.zeros_like(full, dtype=torch.int32)
    for lo, hi in parts:
        mine = torch.zeros_like(full)
        _, ev = rm.pair_matrix(gl, pair_begin=lo, pair_end=hi, out=mine, **kw)
        total += mine
        touched += (mine != 0).int()
        evals += int(ev.item())
    assert torch.equal(total, full)                     # disjoint entries: adding zeros changes no bit
    assert int(touched.max().item()) <= 1               # no entry written by two ranks
    assert evals == int(ev_full.item())
    assert gl.status_flags() == 0


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _nccl_rank(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["NCCL_NVLS_ENABLE"] = "0"
    import torch
    import torch.distributed as dist
    torch.cuda.set_device(rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", rank))
    import paper_2607_16784_b200 as rm
    from paper_2607_16784_b200.shard import pair_matrix_sharded
    lib = rs.make_library(3, num_profiles=48)
    gl = rm.library_build(lib.grid_blocks, lib.block_threads, lib.regs_per_thread, lib.smem_per_block,
                          lib.dur_us, lib.gap_us, lib.offsets, lib.spec)
    Pm, ev = pair_matrix_sharded(gl, rank, world, mode=0, n_align=8, start_filter=1)
    full, ev_full = rm.pair_matrix(gl, mode=0, n_align=8, start_filter=1)
    ok = torch.equal(Pm, full) and int(ev.item()) == int(ev_full.item())
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_two_nccl_ranks_shard_and_combine(tmp_path):
    """Two processes, one GPU each: ranges, NCCL sum all-reduce, every rank ends with the full matrix."""
    torch, _ = _gpu()
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    import torch.multiprocessing as mp
    mp.spawn(_nccl_rank, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert open(tmp_path / f"rank{r}.txt").read() == "ok"
