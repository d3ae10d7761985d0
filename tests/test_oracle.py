"""Pins for the CPU oracle: each test fixes it against something other than itself.

The layer (Section 3.2.2, LoRA): Y = X W^T + s (X A^T) B^T with frozen W and its three
gradients.  A dropped term, a wrong sign, a missing scale or a transposed operand in
oracle/lora_oracle.py fails at least one test here (test_planted_mistakes_are_caught shows it).
"""
import os

import numpy as np
import pytest

from oracle import lora_oracle as oracle
from paper_2503_22673_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "rank1_example.txt")


def _read_golden(path):
    out, name, rows, need = {}, None, [], 0
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if name is None:
                name, need, _ = tok[0], int(tok[1]), int(tok[2])
                rows = []
            else:
                rows.append([float(v) for v in tok])
                if len(rows) == need:
                    out[name] = np.array(rows, dtype=np.float64)
                    name = None
    return out


def _tiny(seed, T=5, d_in=6, d_out=4, r=2):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((T, d_in)), rng.standard_normal((d_out, d_in)),
            rng.standard_normal((r, d_in)), rng.standard_normal((d_out, r)),
            rng.standard_normal((T, d_out)))


# ---------------------------------------------------------------- hand-derived example
def test_hand_derived_rank1_example_is_exact():
    g = _read_golden(GOLDEN)
    s = float(g["s"][0, 0])
    Y = oracle.forward(g["X"], g["W"], g["A"], g["B"], s)
    dX, dA, dB = oracle.backward(g["dY"], g["X"], g["W"], g["A"], g["B"], s)
    assert np.array_equal(Y, g["Y"])
    assert np.array_equal(dX, g["dX"])
    assert np.array_equal(dA, g["dA"])
    assert np.array_equal(dB, g["dB"])


# ---------------------------------------------------------------- brute force, pure Python
def _loops(X, W, A, B, dY, s):
    T, d_in = len(X), len(X[0])
    d_out, r = len(B), len(B[0])
    Y = [[0.0] * d_out for _ in range(T)]
    dX = [[0.0] * d_in for _ in range(T)]
    dA = [[0.0] * d_in for _ in range(r)]
    dB = [[0.0] * r for _ in range(d_out)]
    for o in range(d_out):                      # deliberately o-t-i order, P and Q per element
        for t in range(T):
            acc = 0.0
            for i in range(d_in):
                acc += X[t][i] * W[o][i]
            for j in range(r):
                p = 0.0
                for i in range(d_in):
                    p += X[t][i] * A[j][i]
                acc += s * p * B[o][j]
                dB[o][j] += s * dY[t][o] * p
            Y[t][o] = acc
    for t in range(T):
        for i in range(d_in):
            acc = 0.0
            for o in range(d_out):
                acc += dY[t][o] * W[o][i]
            for j in range(r):
                q = 0.0
                for o in range(d_out):
                    q += dY[t][o] * B[o][j]
                acc += s * q * A[j][i]
                dA[j][i] += s * q * X[t][i]
            dX[t][i] = acc
    return np.array(Y), np.array(dX), np.array(dA), np.array(dB)


@pytest.mark.parametrize("shape", [(5, 6, 4, 2), (3, 7, 5, 1), (1, 2, 3, 3), (4, 1, 1, 2)])
def test_against_pure_python_loops(shape):
    T, d_in, d_out, r = shape
    X, W, A, B, dY = _tiny(11, T, d_in, d_out, r)
    s = 1.7
    Y0, dX0, dA0, dB0 = _loops(X.tolist(), W.tolist(), A.tolist(), B.tolist(), dY.tolist(), s)
    Y = oracle.forward(X, W, A, B, s)
    dX, dA, dB = oracle.backward(dY, X, W, A, B, s)
    for got, ref in ((Y, Y0), (dX, dX0), (dA, dA0), (dB, dB0)):
        assert got.shape == ref.shape
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- finite differences
def test_gradients_by_central_differences():
    X, W, A, B, dY = _tiny(3)
    s, h = 0.75, 1e-3
    dX, dA, dB = oracle.backward(dY, X, W, A, B, s)

    def L(Xv, Av, Bv):
        return float(np.sum(dY * oracle.forward(Xv, W, Av, Bv, s)))

    # L is linear in X, in A (B fixed) and in B (A fixed): central differences are exact
    # up to float64 rounding.
    for name, grad, base in (("X", dX, X), ("A", dA, A), ("B", dB, B)):
        for idx in np.ndindex(base.shape):
            e = np.zeros_like(base)
            e[idx] = h
            args_p = {"X": X, "A": A, "B": B}
            args_m = dict(args_p)
            args_p[name] = base + e
            args_m[name] = base - e
            fd = (L(args_p["X"], args_p["A"], args_p["B"]) - L(args_m["X"], args_m["A"], args_m["B"])) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-8 * max(1.0, abs(grad[idx])), (name, idx, fd, grad[idx])


# ---------------------------------------------------------------- reduction to one dense GEMM
def test_merged_weight_identity():
    X, W, A, B, dY = _tiny(5, T=9, d_in=8, d_out=7, r=3)
    s = 2.0
    Wm = W + s * np.einsum("or,ri->oi", B, A)        # merged weight, built without matmul
    Y = oracle.forward(X, W, A, B, s)
    dX, _, _ = oracle.backward(dY, X, W, A, B, s)
    np.testing.assert_allclose(Y, np.einsum("ti,oi->to", X, Wm), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, np.einsum("to,oi->ti", dY, Wm), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- closed forms
def test_closed_forms_zero_factors():
    X, W, A, B, dY = _tiny(7, T=6, d_in=5, d_out=4, r=2)
    s = 2.0
    base_Y = np.einsum("ti,oi->to", X, W)
    base_dX = np.einsum("to,oi->ti", dY, W)
    # B = 0: adapter contributes nothing to Y/dX and dA vanishes exactly; dB does not.
    Z = np.zeros_like(B)
    assert np.array_equal(oracle.forward(X, W, A, Z, s), X @ W.T)
    np.testing.assert_allclose(oracle.forward(X, W, A, Z, s), base_Y, rtol=1e-13, atol=1e-13)
    dX, dA, dB = oracle.backward(dY, X, W, A, Z, s)
    np.testing.assert_allclose(dX, base_dX, rtol=1e-13, atol=1e-13)
    assert np.all(dA == 0.0)
    assert np.max(np.abs(dB)) > 0.0
    # A = 0: dB vanishes exactly; dA does not.
    ZA = np.zeros_like(A)
    np.testing.assert_allclose(oracle.forward(X, W, ZA, B, s), base_Y, rtol=1e-13, atol=1e-13)
    dX, dA, dB = oracle.backward(dY, X, W, ZA, B, s)
    np.testing.assert_allclose(dX, base_dX, rtol=1e-13, atol=1e-13)
    assert np.all(dB == 0.0)
    assert np.max(np.abs(dA)) > 0.0
    # W = 0: only the rank-r path is left.
    ZW = np.zeros_like(W)
    np.testing.assert_allclose(oracle.forward(X, ZW, A, B, s),
                               s * np.einsum("ti,ji,oj->to", X, A, B), rtol=1e-12, atol=1e-12)


def test_linearity_in_scale():
    X, W, A, B, dY = _tiny(9, T=6, d_in=5, d_out=4, r=2)
    Y0 = oracle.forward(X, W, A, B, 0.0)
    Y1 = oracle.forward(X, W, A, B, 1.0)
    dX0, dA0, dB0 = oracle.backward(dY, X, W, A, B, 0.0)
    dX1, dA1, dB1 = oracle.backward(dY, X, W, A, B, 1.0)
    assert np.all(dA0 == 0.0) and np.all(dB0 == 0.0)
    for s in (0.5, 1.7, 2.0, -3.0):
        Ys = oracle.forward(X, W, A, B, s)
        dXs, dAs, dBs = oracle.backward(dY, X, W, A, B, s)
        np.testing.assert_allclose(Ys - Y0, s * (Y1 - Y0), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(dXs - dX0, s * (dX1 - dX0), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(dAs, s * dA1, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(dBs, s * dB1, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- adjoint identities at benchmark shape
def test_adjoint_identities_on_tiny_workload():
    (p, t), = list(inputs.draw_workload(0, seed=0))
    X, W, A, B, dY = (inputs.bf16_to_f64(t[k]) for k in ("X", "W", "A", "B", "dY"))
    Y = oracle.forward(X, W, A, B, p.scale)
    dX, dA, dB = oracle.backward(dY, X, W, A, B, p.scale)
    assert Y.shape == (p.T, p.d_out) and dX.shape == (p.T, p.d_in)
    assert dA.shape == (p.r, p.d_in) and dB.shape == (p.d_out, p.r)
    lhs, rhs = np.sum(dY * Y), np.sum(dX * X)
    assert abs(lhs - rhs) <= 1e-10 * abs(lhs)
    a, b = np.sum(dA * A), np.sum(dB * B)
    c = np.sum(dY * (Y - np.einsum("ti,oi->to", X, W)))
    assert abs(a - b) <= 1e-10 * abs(a) and abs(a - c) <= 1e-10 * abs(a)


def test_row_independence_and_additivity():
    X, W, A, B, dY = _tiny(13, T=10, d_in=6, d_out=5, r=2)
    s = 2.0
    Y = oracle.forward(X, W, A, B, s)
    dX, dA, dB = oracle.backward(dY, X, W, A, B, s)
    perm = np.random.default_rng(0).permutation(10)
    np.testing.assert_allclose(oracle.forward(X[perm], W, A, B, s), Y[perm], rtol=1e-13, atol=1e-13)
    rows = [7, 0, 3]
    np.testing.assert_allclose(oracle.forward_rows(rows, X, W, A, B, s), Y[rows], rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(oracle.backward_dx_rows(rows, dY, W, A, B, s), dX[rows], rtol=1e-13, atol=1e-13)
    # adapter gradients are sums over token rows: two halves add up to the whole
    h = 4
    _, dA1, dB1 = oracle.backward(dY[:h], X[:h], W, A, B, s)
    _, dA2, dB2 = oracle.backward(dY[h:], X[h:], W, A, B, s)
    np.testing.assert_allclose(dA1 + dA2, dA, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dB1 + dB2, dB, rtol=1e-12, atol=1e-12)
    dA3, dB3 = oracle.backward_adapter_grads(dY, X, A, B, s)
    np.testing.assert_allclose(dA3, dA, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dB3, dB, rtol=1e-13, atol=1e-13)


def test_rel_err_measure():
    ref = np.array([[1.0, -4.0], [2.0, 0.0]])
    assert oracle.rel_err(ref, ref) == 0.0
    assert oracle.rel_err(ref + np.array([[0.0, 0.0], [0.0, 0.2]]), ref) == pytest.approx(0.05)
    assert oracle.rel_err(np.zeros((0, 3)), np.zeros((0, 3))) == 0.0
    with pytest.raises(ValueError):
        oracle.rel_err(np.zeros((2, 2)), np.zeros((2, 3)))


# ---------------------------------------------------------------- dense weight gradient (full fine-tuning)
def test_dense_weight_grad_hand_example_is_exact():
    g = _read_golden(os.path.join(os.path.dirname(__file__), "golden", "dense_dw_example.txt"))
    dW = oracle.dense_weight_grad(g["dY"], g["X"])
    assert np.array_equal(dW, g["dW"])
    assert not np.array_equal(g["X"].T @ g["dY"][:, :2], g["dW"][:2])       # transposed operands are rejected


def test_dense_weight_grad_loops_differences_and_projections():
    X, W, A, B, dY = _tiny(17, T=7, d_in=5, d_out=4, r=2)
    s, h = 1.3, 1e-3
    dW = oracle.dense_weight_grad(dY, X)
    assert dW.shape == W.shape
    # pure-Python loops
    ref = [[sum(dY[t][o] * X[t][i] for t in range(7)) for i in range(5)] for o in range(4)]
    np.testing.assert_allclose(dW, np.array(ref), rtol=1e-12, atol=1e-12)
    # L = <dY, Y(W)> is linear in W: central differences are exact up to rounding
    for idx in np.ndindex(W.shape):
        e = np.zeros_like(W)
        e[idx] = h
        fd = (np.sum(dY * oracle.forward(X, W + e, A, B, s)) - np.sum(dY * oracle.forward(X, W - e, A, B, s))) / (2 * h)
        assert abs(fd - dW[idx]) <= 1e-8 * max(1.0, abs(dW[idx]))
    # the adapter gradients are projections of dW (chain rule through W + s B A)
    _, dA, dB = oracle.backward(dY, X, W, A, B, s)
    np.testing.assert_allclose(s * np.einsum("oj,oi->ji", B, dW), dA, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(s * np.einsum("oi,ji->oj", dW, A), dB, rtol=1e-12, atol=1e-12)
    # sums over token rows: two halves add up
    np.testing.assert_allclose(oracle.dense_weight_grad(dY[:3], X[:3]) + oracle.dense_weight_grad(dY[3:], X[3:]), dW,
                               rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- the pins bite
def test_planted_mistakes_are_caught():
    """Plant plausible mistakes in copies of the oracle formulas (on the CPU) and check that
    the hand-derived example or the loop reference rejects every one of them."""
    g = _read_golden(GOLDEN)
    s = float(g["s"][0, 0])
    X, W, A, B, dY = g["X"], g["W"], g["A"], g["B"], g["dY"]
    wrong_forward = [
        X @ W.T + (X @ A.T) @ B.T,                   # scale dropped
        X @ W.T - s * (X @ A.T) @ B.T,               # sign
        X @ W.T,                                     # adapter dropped
        X @ W.T + s * s * (X @ A.T) @ B.T,           # scale applied twice
    ]
    for cand in wrong_forward:
        assert not np.array_equal(cand, g["Y"])
    Q, P = dY @ B, X @ A.T
    wrong_dx = [dY @ W.T + s * Q @ A, dY @ W + Q @ A, dY @ W, dY @ W - s * Q @ A]
    # W = I in the example hides a transposed W; the loop reference covers that one below.
    for cand in wrong_dx[1:]:
        assert not np.array_equal(cand, g["dX"])
    assert not np.array_equal(P.T @ X * s, g["dA"])          # P used where Q belongs
    assert not np.array_equal(Q.T @ X, g["dA"])              # scale dropped
    assert not np.array_equal(s * dY.T @ Q, g["dB"])         # Q used where P belongs
    assert not np.array_equal(dY.T @ P, g["dB"])             # scale dropped
    Xr, Wr, Ar, Br, dYr = _tiny(21, T=4, d_in=4, d_out=4, r=2)
    Y0, dX0, _, _ = _loops(Xr.tolist(), Wr.tolist(), Ar.tolist(), Br.tolist(), dYr.tolist(), s)
    assert np.max(np.abs(dYr @ Wr.T + s * (dYr @ Br) @ Ar - dX0)) > 1e-3
    assert np.max(np.abs(Xr @ Wr + s * (Xr @ Ar.T) @ Br.T - Y0)) > 1e-3     # W not transposed
