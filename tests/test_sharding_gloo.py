"""The multi-GPU host logic on CPU: two gloo ranks shard rows, compute their slices independently with the CPU
oracle, gather, and agree on a max-over-ranks time.  (The GPU kernels are the same per rank; no exchange step.)"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_18574_b200 import inputs, sharding


def test_row_shard_properties():
    for total in (0, 1, 127, 128, 129, 1000, 4096, 12544, 262144):
        for world in (1, 2, 3, 4, 8):
            covered = 0
            sizes = []
            for r in range(world):
                start, count = sharding.row_shard(total, world, r)
                assert start == covered and count >= 0
                covered += count
                sizes.append(count)
                if count and start + count < total:
                    assert count % 128 == 0
            assert covered == total
            assert max(sizes) - min(sizes) < 256      # at most one block, plus a short last block
    assert sharding.batch_shard(7, 2, 0) == (0, 4) and sharding.batch_shard(7, 2, 1) == (4, 3)
    assert sharding.rank_seed(5, 0) == 5 and sharding.rank_seed(5, 3) == 3005
    assert sharding.whole_job_rate(10.0, 4, 2.0) == pytest.approx(4 * 10.0 / 2e-3)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, ret_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        p = inputs.make_gemm(300, 48, 64, 11, per_channel=1, relu=1, shift_lo=12, shift_hi=18)
        start, count = sharding.row_shard(p.M, world, rank)
        A = np.ascontiguousarray(p.A[start:start + count])
        C = oracle.gemm_i8(A, p.a_rs, 1, p.B, p.b_rs, p.b_cs, p.N, p.bias, p.mult, p.shift, p.per_channel, count, p.N, p.K, p.relu)
        whole = sharding.gather_rows(torch.from_numpy(C), p.M, world)
        full = oracle.gemm_i8(p.A, p.a_rs, 1, p.B, p.b_rs, p.b_cs, p.N, p.bias, p.mult, p.shift, p.per_channel, p.M, p.N, p.K, p.relu)
        ok = bool(np.array_equal(whole.numpy(), full))
        mx = sharding.max_over_ranks(10.0 + rank)          # rank r "took" 10 + r ms
        ok = ok and mx == 10.0 + (world - 1)
        with open(os.path.join(ret_dir, f"rank{rank}.txt"), "w") as f:
            f.write("ok" if ok else "bad")
    finally:
        dist.destroy_process_group()


def test_two_rank_sharded_gemm_matches_unsharded(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)   # spawn, never fork
    for r in range(world):
        assert (tmp_path / f"rank{r}.txt").read_text() == "ok"
