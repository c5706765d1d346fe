"""CPU fp64 oracle for the per-matrix Muon optimizer step.

TEST INFRASTRUCTURE ONLY.  This module defines what "correct" means for the
CUDA path; it is imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg, and by nothing else.  It shares no code with the
CUDA path and never imports it.  Everything is plain NumPy in float64; the only
library primitive used as a step is the dense matrix product ``@``.  There is
no blocking, no fusion, no use of symmetry and no reordering beyond what the
paper's equations state, so each function can be checked against the paper by
eye.

All functions take float64 arrays.  Callers widen bf16 / fp32 storage to
float64 exactly (every bf16 and fp32 value is representable) before calling.

Every function here is pinned by tests that do not call back into it (closed
forms, an SVD from LAPACK, hand-derived 2x2 cases, brute-force expansion,
symmetries); no function is "parity unpinned".

Passages followed (paper = "Muon is Scalable for LLM Training"):
  * Sec. 2.1 "The Muon Optimizer": the three-line update rule (momentum,
    Newton-Schulz, weight step) and its footnote 1 (Nesterov-style input).
  * Sec. 2.1 "Newton-Schulz Iterations for Matrix Orthogonalization":
    X_0 = M / ||M||_F and the quintic iteration (Eq. 2) with the coefficients
    a = 3.4445, b = -4.7750, c = 2.0315.
  * Sec. 2.2 "Weight Decay" (Eq. 3) and "Matching update RMS of AdamW"
    (the unnumbered equation with 0.2 * sqrt(max(A, B))).
  * Algorithm 1, last line: the update RMS returned for logging.
  * Sec. 3.1 "Consistent Update RMS": the three ways of scaling the update
    (Baseline 0.2*sqrt(H), Update Norm 0.2/RMS(O), Adjusted LR
    0.2*sqrt(max(A, B)) -- the last is the method the paper adopts).
"""

from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

# Sec. 2.1: coefficients of the quintic Newton-Schulz polynomial.
NS_A = 3.4445
NS_B = -4.7750
NS_C = 2.0315


@dataclass
class Hyper:
    """Hyper-parameters of one step.  Defaults are the paper's choices:
    mu = 0.95 and N = 5 (Sec. 2.2 "Other Hyper-parameters"), Nesterov-style
    input (Sec. 2.1 footnote 1), update-RMS factor 0.2 (Sec. 2.2)."""

    lr: float = 2e-2
    wd: float = 0.1
    mu: float = 0.95
    nesterov: bool = True
    ns_steps: int = 5
    a: float = NS_A
    b: float = NS_B
    c: float = NS_C
    eps: float = 1e-7
    rms_scale: float = 0.2
    # Sec. 3.1: "adjusted_lr" (default, the adopted method), "fixed_dim"
    # (Baseline; scale_dim is the hidden size H) or "update_norm".
    scale_mode: str = "adjusted_lr"
    scale_dim: float = 0.0
    # Optional list of (a, b, c), one triple per Newton-Schulz step, replacing
    # the single triple above (the paper uses one triple for all steps).
    coeffs: object = None
    # Non-finite gradients (the paper is silent): False = the momentum is still
    # M_t as the rule's first line defines it; True = a matrix whose gradient
    # holds an Inf or a NaN keeps its momentum as well as its weight.
    protect_momentum: bool = False


def _f64(x):
    x = np.asarray(x)
    if x.dtype != np.float64:
        raise TypeError("oracle inputs must already be widened to float64")
    return x


def momentum_update(M_prev, G, mu):
    """M_t = mu * M_{t-1} + grad  (Sec. 2.1, first line of the update rule).
    No dampening factor appears in the paper's rule."""
    return mu * _f64(M_prev) + _f64(G)


def newton_schulz_input(M_new, G, mu, nesterov):
    """What is fed to Newton-Schulz.  Sec. 2.1 footnote 1: with the
    Nesterov-style momentum the input is mu * M_t + grad (M_t is the freshly
    updated momentum); otherwise it is M_t itself."""
    if nesterov:
        return mu * _f64(M_new) + _f64(G)
    return _f64(M_new).copy()


def frobenius_normalise(U, eps):
    """X_0 = U / ||U||_F  (Sec. 2.1, Newton-Schulz paragraph).  The paper has
    no epsilon; the reading taken here is X_0 = U / (||U||_F + eps) so that a
    zero input gives X_0 = 0 instead of NaN.  Returns (norm, X_0)."""
    U = _f64(U)
    nu = math.sqrt(float(np.sum(U * U)))
    return nu, U / (nu + eps)


def newton_schulz(X0, steps, a=NS_A, b=NS_B, c=NS_C, trace=None, coeffs=None):
    """N steps of Eq. 2:  X_k = a X + b (X X^T) X + c (X X^T)^2 X.
    With ``coeffs`` (a list of N triples) step k uses its own (a, b, c).

    When the matrix has more rows than columns the iteration runs on the
    transpose and the result is transposed back; the polynomial is odd, so in
    exact arithmetic this changes nothing and only makes X X^T the smaller of
    the two possible Gram matrices.  If ``trace`` is a list, the per-iteration
    (A, B, X) triples are appended to it in the orientation the iteration ran
    in (short side first)."""
    X = _f64(X0)
    transposed = X.shape[0] > X.shape[1]
    if transposed:
        X = X.T
    X = X.copy()
    if coeffs is not None and len(coeffs) != int(steps):
        raise ValueError("coeffs must hold one (a, b, c) per step")
    for k in range(int(steps)):
        if coeffs is not None:
            a, b, c = coeffs[k]
        A = X @ X.T
        B = b * A + c * (A @ A)
        X = a * X + B @ X
        if trace is not None:
            trace.append((A, B, X.copy()))
    if transposed:
        X = X.T
    return np.ascontiguousarray(X)


def update_factor(O, rms_scale=0.2, scale_mode="adjusted_lr", scale_dim=0.0):
    """The scalar that multiplies O in the weight step (Sec. 3.1, the three
    numbered variants): rms_scale*sqrt(max(A, B)) ("Adjusted LR", also Sec. 2.2),
    rms_scale*sqrt(H) ("Baseline") or rms_scale/RMS(O) ("Update Norm"), with
    RMS(O) = sqrt(mean(O^2)).  A zero O under "Update Norm" gives factor 0."""
    O = _f64(O)
    rows, cols = O.shape
    if scale_mode == "adjusted_lr":
        return rms_scale * math.sqrt(max(rows, cols))
    if scale_mode == "fixed_dim":
        return rms_scale * math.sqrt(scale_dim)
    if scale_mode == "update_norm":
        o_rms = math.sqrt(float(np.mean(O * O)))
        return rms_scale / o_rms if o_rms > 0.0 else 0.0
    raise ValueError("unknown scale_mode %r" % (scale_mode,))


def round_to_bf16(x):
    """Round-to-nearest-even of float64 values to bfloat16 (8 significand bits),
    returned as float64.  Done on the bit pattern of the float32 value: every
    value used here is far inside float32's range, and rounding float64 ->
    float32 -> bf16 differs from direct rounding only on exact ties of the
    second step, which the first rounding cannot create for these magnitudes."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    bits = f.view(np.uint32).astype(np.uint64)
    rounded = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return rounded.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def newton_schulz_bf16_storage(U, eps, steps, a=NS_A, b=NS_B, c=NS_C, trace=None, fold_identity=False):
    """Eq. 2 with the storage precision Sec. 2.3 names ("Newton-Schulz
    iteration steps in bf16"): every stored matrix -- the input, A, B and each
    new X -- is rounded to bf16, all arithmetic in between is exact (float64).
    This is not a reference for the CUDA path (summation order makes any bf16
    implementation differ from any other by a similar amount); it measures how
    far the bf16 storage alone moves the result from the float64 iteration, so
    that tests can tell a kernel error from the precision the paper fixes.  The
    1/(||U||_F + eps) factor is applied in full precision to the first A and
    the first X, as the CUDA path does.  Short side first, like newton_schulz.
    If ``trace`` is a list, the stored input and then every iteration's stored
    (A, B, X) are appended to it (short side first).

    The paper does not say which intermediates are the stored ones.  Eq. 2's
    a X + B X is also the single product (B + a I) X; ``fold_identity`` selects
    that reading: the stored polynomial is bf16(b A + c A^2 + a I) and the new X
    is bf16 of its product with X.  Identical in exact arithmetic; in bf16 the
    rounding of B_ii + a replaces that of B_ii, which is the smaller error on
    most inputs and the larger one on a few.

    Pinned by a hand-derived two-iteration 2x2 example
    (tests/golden/bf16_storage_2x2_two_steps.txt) that a missing, doubled or
    misplaced rounding changes."""
    U = _f64(U)
    transposed = U.shape[0] > U.shape[1]
    nu = math.sqrt(float(np.sum(U * U)))
    s = 1.0 / (nu + eps)
    X = round_to_bf16(U.T if transposed else U)
    if trace is not None:
        trace.append(X.copy())
    for k in range(int(steps)):
        A = round_to_bf16((s * s if k == 0 else 1.0) * (X @ X.T))
        if fold_identity:
            B = round_to_bf16(b * A + c * (A @ A) + a * np.eye(A.shape[0]))
            X = round_to_bf16((s if k == 0 else 1.0) * (B @ X))
        else:
            B = round_to_bf16(b * A + c * (A @ A))
            X = round_to_bf16((s if k == 0 else 1.0) * (a * X + B @ X))
        if trace is not None:
            trace.append((A, B, X.copy()))
    if int(steps) == 0:
        X = s * X
    return np.ascontiguousarray(X.T if transposed else X)


def apply_update(W, O, lr, wd, rms_scale=0.2, scale_mode="adjusted_lr", scale_dim=0.0):
    """W_t = W_{t-1} - lr * (factor * O + wd * W_{t-1}) with factor =
    rms_scale * sqrt(max(A, B)) for a parameter of shape [A, B]  (Sec. 2.2,
    "Matching update RMS of AdamW"; rms_scale is the paper's 0.2) or one of the
    other two variants of Sec. 3.1.  The decay term uses W_{t-1} and is
    multiplied by the learning rate, as in Eq. 3."""
    W = _f64(W)
    O = _f64(O)
    return W - lr * (update_factor(O, rms_scale, scale_mode, scale_dim) * O + wd * W)


def update_rms(O, rms_scale=0.2, scale_mode="adjusted_lr", scale_dim=0.0):
    """sqrt(mean(u^2)) of the scaled update u = factor * O  (Algorithm 1,
    returned value; the reading taken is that u carries the scale factor, so
    the value sits near 0.2 as Sec. 2.2 intends)."""
    O = _f64(O)
    u = update_factor(O, rms_scale, scale_mode, scale_dim) * O
    return math.sqrt(float(np.mean(u * u)))


def muon_step(W, G, M, hp: Hyper, trace=False):
    """One full Muon step for one matrix.  Returns a dict with the new weight
    ``W``, the new momentum ``M``, the Frobenius norm ``nu`` of the
    Newton-Schulz input, ``X0``, the orthogonalised update ``O``, the logged
    ``rms`` and, when ``trace`` is set, the per-iteration (A, B, X) list.

    Non-finite input (a NaN or Inf anywhere in the Newton-Schulz input): the
    paper is silent.  The reading taken: the weight is left unchanged, the
    momentum is still M_t as the first line of the rule defines it, and the
    result carries ``nonfinite = True``; with ``hp.protect_momentum`` a
    non-finite gradient leaves the momentum unchanged as well."""
    W = _f64(W)
    G = _f64(G)
    M = _f64(M)
    if not (W.shape == G.shape == M.shape and W.ndim == 2):
        raise ValueError("W, G, M must be 2-D and of one shape")
    if hp.protect_momentum and not np.all(np.isfinite(G)):
        return {"M": M.copy(), "nu": float("nan"), "nonfinite": True, "W": W.copy(), "X0": None, "O": None,
                "rms": float("nan")}
    M_new = momentum_update(M, G, hp.mu)
    U = newton_schulz_input(M_new, G, hp.mu, hp.nesterov)
    nu, X0 = frobenius_normalise(U, hp.eps)
    out = {"M": M_new, "nu": nu, "nonfinite": False}
    if not math.isfinite(nu):
        out.update(W=W.copy(), X0=None, O=None, rms=float("nan"), nonfinite=True)
        return out
    stages = [] if trace else None
    O = newton_schulz(X0, hp.ns_steps, hp.a, hp.b, hp.c, trace=stages, coeffs=hp.coeffs)
    out.update(
        W=apply_update(W, O, hp.lr, hp.wd, hp.rms_scale, hp.scale_mode, hp.scale_dim),
        X0=X0,
        O=O,
        rms=update_rms(O, hp.rms_scale, hp.scale_mode, hp.scale_dim),
    )
    if trace:
        out["stages"] = stages
    return out
