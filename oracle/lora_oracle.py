"""CPU oracle for the LoRA projection layer, forward and backward.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this file; it exists so
that the CUDA kernels can be compared against the plain definition.  It shares no code
with the CUDA library.

The layer (Section 3.2.2, "LoRA (Low-Rank Adaptation)", Hu et al. 2021; adapter
hyper-parameters r and alpha from Section 4.5, scale s = alpha / r) with frozen W is

    forward    Y  = X W^T + s (X A^T) B^T
    backward   dX = dY W + s (dY B) A
               dB = s dY^T (X A^T)
               dA = s (dY B)^T X

with X[T, d_in], W[d_out, d_in], A[r, d_in], B[d_out, r], dY[T, d_out].  The result is
exact linear algebra, so the oracle is the definition itself, evaluated in float64 on the
exactly widened inputs with no intermediate rounding.  numpy's float64 matmul serves as
the contraction primitive; there is no blocking or fusion here.

Pins (tests/test_oracle.py): a hand-derived rank-1 example stored under tests/golden/,
pure-Python triple loops on tiny inputs, central finite differences of L = <dY, Y>,
the merged-weight identity Y = X (W + s B A)^T, the closed forms for B = 0 / A = 0 / W = 0,
linearity in s, and the adjoint identities <dY,Y> = <dX,X>, <dA,A> = <dB,B>.
Every function here has at least one such pin; none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


def forward(X, W, A, B, s: float) -> np.ndarray:
    """Y = X W^T + s (X A^T) B^T  (LoRA forward, Section 3.2.2)."""
    X, W, A, B = _f64(X), _f64(W), _f64(A), _f64(B)
    P = X @ A.T                      # [T, r]
    return X @ W.T + float(s) * (P @ B.T)


def backward(dY, X, W, A, B, s: float):
    """(dX, dA, dB) for frozen W (LoRA backward, Section 3.2.2).

    dX = dY W + s (dY B) A ;  dA = s (dY B)^T X ;  dB = s dY^T (X A^T)
    """
    dY, X, W, A, B = _f64(dY), _f64(X), _f64(W), _f64(A), _f64(B)
    s = float(s)
    P = X @ A.T                      # [T, r]
    Q = dY @ B                       # [T, r]
    dX = dY @ W + s * (Q @ A)
    dA = s * (Q.T @ X)
    dB = s * (dY.T @ P)
    return dX, dA, dB


def forward_rows(rows, X, W, A, B, s: float) -> np.ndarray:
    """Rows ``rows`` of Y.  Token rows are independent, so this is ``forward`` on X[rows]."""
    return forward(_f64(X)[np.asarray(rows)], W, A, B, s)


def backward_dx_rows(rows, dY, W, A, B, s: float) -> np.ndarray:
    """Rows ``rows`` of dX = dY W + s (dY B) A (each row depends only on its own dY row)."""
    dYr = _f64(dY)[np.asarray(rows)]
    W, A, B = _f64(W), _f64(A), _f64(B)
    return dYr @ W + float(s) * ((dYr @ B) @ A)


def backward_adapter_grads(dY, X, A, B, s: float):
    """(dA, dB) alone; W does not enter them."""
    dY, X, A, B = _f64(dY), _f64(X), _f64(A), _f64(B)
    s = float(s)
    dA = s * ((dY @ B).T @ X)
    dB = s * (dY.T @ (X @ A.T))
    return dA, dB


def dense_weight_grad(dY, X) -> np.ndarray:
    """dW = dY^T X, the gradient of L = <dY, X W^T> with respect to W itself.

    This is the extra contraction full fine-tuning pays for and LoRA avoids (Section 4.5,
    "Full-model tuning": every weight is updated).  dW[o, i] = sum_t dY[t, o] X[t, i].
    Pins (tests/test_oracle.py): a hand-derived small example under tests/golden/, Python loops,
    central differences of L in W, and the two projections dA = s B^T dW, dB = s dW A^T that
    tie it to the adapter gradients above.
    """
    return _f64(dY).T @ _f64(X)


def rel_err(got, ref) -> float:
    """max|got - ref| / max|ref|  (the agreement measure; 0/0 counts as 0)."""
    got, ref = _f64(got), _f64(ref)
    if got.shape != ref.shape:
        raise ValueError(f"shape mismatch {got.shape} vs {ref.shape}")
    if ref.size == 0:
        return 0.0
    num = float(np.max(np.abs(got - ref)))
    den = float(np.max(np.abs(ref)))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den
