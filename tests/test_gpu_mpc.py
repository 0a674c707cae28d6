"""GPU parity of the TinyMPC forward pass (fp32) against the fp64 oracle.

Tolerance.  Each output is a chain of at most nhorizon dot products of 12 to 16 fused multiply-adds in fp32
(unit round-off 2^-24); a dot product of n terms carries a relative error of about n * 2^-24 of the sum of its
absolute terms, and the recurrence multiplies earlier errors by at most the row sums of |Adyn - Bdyn Kinf|
(below 2 for the stable stand-in systems used here).  With |x|, |u| of order 1..4 over five steps that bounds
the absolute error by roughly 5 * 2^4 * 16 * 2^-24 * 4 < 4e-4; the test allows 1e-4 * (1 + max |u|), and the
observed error is near 1e-6.
"""
import numpy as np
import pytest

from paper_2505_18574_b200 import inputs

pytestmark = pytest.mark.gpu


def _run(p, states=False):
    import torch
    import paper_2505_18574_b200 as i8
    x0 = torch.from_numpy(p.x0).cuda(); d = torch.from_numpy(p.d).cuda()
    u = torch.full((p.batch, p.nhorizon, 4), float("nan"), dtype=torch.float32, device="cuda")
    xs = torch.full((p.batch, p.nhorizon, 12), float("nan"), dtype=torch.float32, device="cuda") if states else None
    i8.mpc_forward_f32(p.Adyn, p.Bdyn, p.Kinf, x0, d, u, xs)
    torch.cuda.synchronize()
    return u.cpu().numpy(), (xs.cpu().numpy() if states else None)


# horizons up to 5 stream chunks of 256 instances, up to 14 chunks of 128, longer ones take one thread per instance;
# 300000 and 700001 instances give every persistent CTA several rounds (ring slots refilled, barrier phases flipping)
@pytest.mark.parametrize("batch,nh", [(1, 5), (7, 5), (256, 5), (1000, 1), (4099, 8), (100000, 5), (129, 9), (3000, 12),
                                      (300000, 5), (700001, 3), (150000, 14), (2000, 20), (257, 5), (255, 2)])
def test_mpc_forward_matches_oracle(batch, nh):
    import oracle
    p = inputs.make_mpc(batch, nh, seed=40 + nh)
    want_u, want_x = oracle.mpc_forward(p.Adyn, p.Bdyn, p.Kinf, p.x0, p.d, return_states=True)
    got_u, got_x = _run(p, states=True)
    tol = 1e-4 * (1.0 + np.abs(want_u).max())
    assert np.isfinite(got_u).all() and np.isfinite(got_x).all()
    assert np.abs(got_u - want_u).max() <= tol, np.abs(got_u - want_u).max()
    assert np.abs(got_x - want_x).max() <= 1e-4 * (1.0 + np.abs(want_x).max())
    got_u2, _ = _run(p, states=False)                 # the states are optional
    assert np.array_equal(got_u2, got_u)


def test_mpc_closed_form_on_gpu():
    """Oracle-independent: with Kinf = 0 the output is exactly -d, and the hand-worked example of the golden file."""
    import os
    p = inputs.make_mpc(513, 5, seed=3)
    p.Kinf[:] = 0
    got, _ = _run(p)
    assert np.array_equal(got, -p.d)
    rows = [list(map(float, l.split())) for l in open(os.path.join(os.path.dirname(__file__), "golden", "mpc_forward_worked.txt"))
            if l.strip() and not l.startswith("#")]
    q = inputs.make_mpc(2, 3, seed=1)
    q.Adyn[:] = np.eye(12); q.Bdyn[:] = 0; q.Bdyn[:4] = np.eye(4); q.Kinf[:] = 0; q.Kinf[:, :4] = np.eye(4)
    q.x0[:] = np.arange(1, 13); q.d[:] = np.array([0.5, 0, 0, -1.0])
    got, _ = _run(q)
    assert np.array_equal(got[0], np.array(rows, dtype=np.float32)) and np.array_equal(got[1], got[0])


def test_mpc_argument_validation():
    import paper_2505_18574_b200 as i8
    L = i8.lib()
    assert L.mpc_forward_f32(None, None, None, None, None, None, None, -1, 5, None) == 2
    assert L.mpc_forward_f32(None, None, None, None, None, None, None, 4, 5, None) == 1
    assert L.mpc_forward_f32(None, None, None, None, None, None, None, 0, 5, None) == 0
