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


# Host implementations with the binding's signatures, built on the oracle: they let the sharded wrappers (slicing,
# launching on the local slice, gathering) run on CPU ranks.
def _host_gemm(A, B, C, bias, mult, shift, per_channel, relu):
    import oracle
    a = np.ascontiguousarray(A.numpy()); bt = np.ascontiguousarray(B.t().numpy())      # B view (K, N) -> storage (N, K)
    M, K = a.shape
    N = bt.shape[0]
    C.copy_(torch.from_numpy(oracle.gemm_i8(a, K, 1, bt, 1, K, N, None if bias is None else bias.numpy(), mult.numpy(), shift.numpy(),
                                            per_channel, M, N, K, relu)))


def _host_conv(x, w, y, bias, mult, shift, per_channel, relu, stride, pad):
    import oracle
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    y.copy_(torch.from_numpy(oracle.conv2d_i8(np.ascontiguousarray(x.numpy()), w.numpy(), bias.numpy(), mult.numpy(), shift.numpy(),
                                              per_channel, N, H, W, C, K, R, S, stride[0], stride[1], pad[0], pad[1], relu)))


def _host_batched(A, B, C, bias, mult, shift, per_channel, relu):
    import oracle
    batch, M, K = A.shape
    N = B.shape[2]
    b = None if bias is None else np.ascontiguousarray(bias.numpy())
    out = oracle.batched_gemm_i8(np.ascontiguousarray(A.numpy()), K, 1, M * K, np.ascontiguousarray(B.numpy()), N, 1, K * N, N, M * N,
                                 b, N if (b is not None and b.ndim == 2) else 0, mult.numpy(), shift.numpy(), per_channel, batch, M, N, K, relu)
    C.copy_(torch.from_numpy(out.reshape(batch, M, N)))


def _sharded_wrappers_agree(world, rank):
    """Every rank calls the wrappers on the whole problem; the gathered results must equal the unsharded ones."""
    import oracle
    T = torch.from_numpy
    g = inputs.make_gemm(700, 40, 48, 21, per_channel=1, relu=0, shift_lo=12, shift_hi=18)
    whole = sharding.sharded_gemm_i8(T(g.A), T(g.B).t(), T(g.bias), T(g.mult), T(g.shift), 1, 0, gather=True, kernel=_host_gemm)
    ok = np.array_equal(whole.numpy(), oracle.gemm_i8(g.A, g.K, 1, g.B, 1, g.K, g.N, g.bias, g.mult, g.shift, 1, g.M, g.N, g.K, 0))
    local = sharding.sharded_gemm_i8(T(g.A), T(g.B).t(), T(g.bias), T(g.mult), T(g.shift), 1, 0, kernel=_host_gemm)
    start, count = sharding.row_shard(g.M, world, rank)
    ok = ok and local.shape[0] == count and np.array_equal(local.numpy(), whole.numpy()[start:start + count])
    c = inputs.make_conv(5, 9, 8, 8, 6, 3, 3, 2, 1, 22)
    y = sharding.sharded_conv2d_i8(T(c.x), T(c.w), T(c.bias), T(c.mult), T(c.shift), 1, 1, (2, 2), (1, 1), gather=True, kernel=_host_conv)
    ok = ok and np.array_equal(y.numpy(), oracle.conv2d_i8(c.x, c.w, c.bias, c.mult, c.shift, 1, c.N, c.H, c.W, c.C, c.K, 3, 3, 2, 2, 1, 1, 1))
    b = inputs.make_batched(7, 16, 16, 16, 23)
    cb = sharding.sharded_batched_gemm_i8(T(b.A), T(b.B), T(b.bias), T(b.mult), T(b.shift), 0, 1, gather=True, kernel=_host_batched)
    want = oracle.batched_gemm_i8(b.A, 16, 1, 256, b.B, 16, 1, 256, 16, 256, b.bias, 16, b.mult, b.shift, 0, 7, 16, 16, 16, 1).reshape(7, 16, 16)
    return bool(ok and np.array_equal(cb.numpy(), want))


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
        ok = ok and _sharded_wrappers_agree(world, rank)
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
