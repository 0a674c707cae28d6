"""Pins for the oracle's TinyMPC forward pass (CPU only): a hand-worked example, closed forms, numpy's
matrix routines, and planted mistakes that the pins must catch."""
import os
import subprocess
import tempfile

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(os.path.dirname(HERE), "oracle", "oracle.c")


def _rand(seed, batch=3, nh=5):
    rng = np.random.default_rng(seed)
    return (np.eye(12) + 0.1 * rng.standard_normal((12, 12)), rng.standard_normal((12, 4)), rng.standard_normal((4, 12)),
            rng.standard_normal((batch, 12)), rng.standard_normal((batch, nh, 4)))


def pin_worked_example(O):
    rows = [list(map(float, l.split())) for l in open(os.path.join(HERE, "golden", "mpc_forward_worked.txt"))
            if l.strip() and not l.startswith("#")]
    A = np.eye(12); B = np.zeros((12, 4)); B[:4] = np.eye(4); K = np.zeros((4, 12)); K[:, :4] = np.eye(4)
    x0 = np.arange(1, 13, dtype=float)[None]; d = np.tile(np.array([0.5, 0, 0, -1.0]), (1, 3, 1))
    u = O.mpc_forward(A, B, K, x0, d)
    assert np.array_equal(u[0], np.array(rows))


def pin_numpy_recurrence(O):
    A, B, K, x0, d = _rand(1)
    u, xs = O.mpc_forward(A, B, K, x0, d, return_states=True)
    for b in range(x0.shape[0]):
        x = x0[b].copy()
        for i in range(d.shape[1]):
            assert np.allclose(xs[b, i], x, rtol=1e-13, atol=1e-13)
            ui = -(K @ x) - d[b, i]
            assert np.allclose(u[b, i], ui, rtol=1e-13, atol=1e-13)
            x = A @ x + B @ ui


def pin_closed_forms(O):
    A, B, K, x0, d = _rand(2)
    # no feedback: u[i] = -d[i] exactly
    assert np.array_equal(O.mpc_forward(A, B, np.zeros((4, 12)), x0, d), -d)
    # no input matrix and no d: x[i] = A^i x0, u[i] = -K A^i x0
    u, xs = O.mpc_forward(A, np.zeros((12, 4)), K, x0, np.zeros_like(d), return_states=True)
    for i in range(d.shape[1]):
        Ai = np.linalg.matrix_power(A, i)
        assert np.allclose(xs[:, i], x0 @ Ai.T, rtol=1e-12, atol=1e-12)
        assert np.allclose(u[:, i], -(x0 @ Ai.T) @ K.T, rtol=1e-12, atol=1e-12)
    # closed loop: x[i+1] = (A - B K) x[i] - B d[i]
    u, xs = O.mpc_forward(A, B, K, x0, d, return_states=True)
    for i in range(d.shape[1] - 1):
        assert np.allclose(xs[:, i + 1], xs[:, i] @ (A - B @ K).T - d[:, i] @ B.T, rtol=1e-12, atol=1e-12)
    # linear in (x0, d); instances are independent
    u2 = O.mpc_forward(A, B, K, 2 * x0, 2 * d)
    assert np.allclose(u2, 2 * u, rtol=1e-12, atol=1e-12)
    perm = np.array([2, 0, 1])
    assert np.array_equal(O.mpc_forward(A, B, K, x0[perm], d[perm]), u[perm])


PINS = [pin_worked_example, pin_numpy_recurrence, pin_closed_forms]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_mpc_oracle_meets_pin(pin):
    pin(oracle.lib())


MUTANTS = [
    ("d_added", "ui[r] = -kx - di[r];", "ui[r] = -kx + di[r];"),
    ("feedback_sign", "ui[r] = -kx - di[r];", "ui[r] = kx - di[r];"),
    ("input_term_dropped", "xn[r] = ax + bu;", "xn[r] = ax;"),
    ("kinf_transposed", "kx += Kinf[r * MPC_NX + c] * x[c];", "kx += Kinf[c * MPC_NU + r] * x[c];"),
    ("adyn_transposed", "ax += Adyn[r * MPC_NX + c] * x[c];", "ax += Adyn[c * MPC_NX + r] * x[c];"),
    ("bdyn_wrong_stride", "bu += Bdyn[r * MPC_NU + c] * ui[c];", "bu += Bdyn[c * MPC_NX + r] * ui[c];"),
    ("state_updated_in_place", "xn[r] = ax + bu;", "xn[r] = ax + bu; x[r] = xn[r];"),
    ("d_not_advanced", "const double *di = d + ((int64_t)b * nhorizon + i) * MPC_NU;", "const double *di = d + ((int64_t)b * nhorizon) * MPC_NU;"),
]


@pytest.mark.parametrize("label,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mpc_pins_catch_planted_mistake(label, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1
    with tempfile.TemporaryDirectory() as dd:
        src = os.path.join(dd, "m.c"); so = os.path.join(dd, "m.so")
        open(src, "w").write(text.replace(old, new))
        subprocess.run(["gcc", "-O1", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", so, src, "-lm"], check=True)
        mutant = oracle.Oracle(so)
        caught = []
        for pin in PINS:
            try:
                pin(mutant)
            except AssertionError:
                caught.append(pin.__name__)
        assert caught, f"no pin noticed '{label}'"
