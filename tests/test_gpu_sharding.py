"""The sharded wrappers on one GPU: world = 1 through the library, and a simulated world of two ranks (both slices
computed on this GPU one after the other and concatenated) against the unsharded oracle result."""
import numpy as np
import pytest

from paper_2505_18574_b200 import inputs, sharding
import harness as H

pytestmark = pytest.mark.gpu


def _t(a):
    import torch
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("world", [1, 2, 3])
def test_sharded_gemm(world):
    import torch
    p = inputs.make_gemm(1000, 320, 256, 31, per_channel=1, relu=1, shift_lo=12, shift_hi=20)
    want = H.gemm_oracle(p)
    A, B = _t(p.A), _t(p.B)
    parts = [sharding.sharded_gemm_i8(A, B.t(), _t(p.bias), _t(p.mult), _t(p.shift), 1, 1, world=world, rank=r) for r in range(world)]
    assert [x.shape[0] for x in parts] == [sharding.row_shard(p.M, world, r)[1] for r in range(world)]
    H.assert_same(torch.cat(parts).cpu().numpy(), want, f"sharded gemm world {world}")


@pytest.mark.parametrize("world", [1, 2])
def test_sharded_conv_and_batched(world):
    import torch
    c = inputs.make_conv(6, 14, 14, 64, 96, 3, 3, 1, 1, 32)
    parts = [sharding.sharded_conv2d_i8(_t(c.x), _t(c.w), _t(c.bias), _t(c.mult), _t(c.shift), 1, 1, (1, 1), (1, 1), world=world, rank=r)
             for r in range(world)]
    H.assert_same(torch.cat(parts).cpu().numpy(), H.conv_oracle(c), f"sharded conv world {world}")
    b = inputs.make_batched(37, 64, 64, 64, 33)
    parts = [sharding.sharded_batched_gemm_i8(_t(b.A), _t(b.B), _t(b.bias), _t(b.mult), _t(b.shift), 0, 1, world=world, rank=r)
             for r in range(world)]
    H.assert_same(torch.cat(parts).cpu().numpy(), H.batched_oracle(b), f"sharded batched world {world}")
