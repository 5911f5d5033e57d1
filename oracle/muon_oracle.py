"""CPU oracle for the layout-driven Muon step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the hot path computes, written
from the paper's statement of the method.  It shares no code with the CUDA library
and must never be imported by the product path; only the tests, the smoke check and
the benchmark's CPU-baseline leg may call it.

Arithmetic is numpy float64 throughout.  `np.matmul` (a library primitive) is the
only non-trivial step; there is no blocking, fusion or reordering beyond what the
algorithm states.  The optional "bf16" mode rounds the declared intermediates
(the staged momentum U and every produced A, B, X) once each to bfloat16, with the
products themselves still accumulated in float64.

Parity status: every function here is pinned by tests that do not re-use its own
formulae (SVD closed form, scalar recurrences, brute-force index maps, invariants),
except the per-step coefficient variant the paper names as its default (an asymmetric
five-step set): the paper prints no values for it, so that variant is *parity
unpinned* beyond the generic per-step-coefficient plumbing.

Notation follows the paper: W (m x n) weight, G gradient, M momentum, X_k the NS
iterate, A = X X^T the Gram factor, (a_k, b_k, c_k) the per-step coefficients.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

# --------------------------------------------------------------------------- bf16 rounding

_BF16_MAX = float.fromhex("0x1.FEp127")          # largest finite bfloat16
_BF16_MIN_EXP = -125                              # frexp exponent of the smallest normal (2**-126 = 0.5 * 2**-125)


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (ties to even); result held as float64.

    bfloat16 keeps 8 significant bits (1 implicit + 7 stored) over the float32 exponent
    range.  A value x = f * 2**e with 0.5 <= |f| < 1 therefore sits on a grid of spacing
    2**(e-8); below the normal range the grid spacing stays 2**-133.  Values that round
    past the largest finite bfloat16 become infinite.
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    q = np.maximum(e, _BF16_MIN_EXP) - 8
    y = np.ldexp(np.rint(np.ldexp(x, -q)), q)      # np.rint rounds half to even
    y = np.where(np.abs(y) > _BF16_MAX, np.copysign(np.inf, x), y)
    y = np.where(np.isfinite(x), y, x)             # inf / nan pass through
    return y


def _round(x: np.ndarray, mode: str) -> np.ndarray:
    if mode == "bf16":
        return bf16_rne(x)
    if mode == "fp64":
        return x
    raise ValueError(f"unknown mode {mode!r}")


# --------------------------------------------------------------------------- flat-shard layout (Sections 5.1-5.2, 6.4)
# A layout is: shapes [(m, n)], and segments [(matrix, elem_begin, elem_count, flat_offset)].
# Segment k says: elements [elem_begin, elem_begin + elem_count) of the row-major
# linearisation of matrix `matrix` live at flat[flat_offset : flat_offset + elem_count].
# Everything else in the flat buffer is padding.


def materialize(flat: np.ndarray, shapes: Sequence[Tuple[int, int]], segments) -> List[np.ndarray]:
    """Unpack the flat shard buffer into whole row-major matrices (the gather's copy-out)."""
    mats = [np.zeros(m * n, dtype=flat.dtype) for (m, n) in shapes]
    for (mat, eb, ec, off) in segments:
        mats[mat][eb:eb + ec] = flat[off:off + ec]
    return [v.reshape(shapes[i]) for i, v in enumerate(mats)]


def scatter(flat: np.ndarray, shapes: Sequence[Tuple[int, int]], segments, matrices: Sequence[np.ndarray]) -> np.ndarray:
    """Pack whole matrices back into (a copy of) the flat shard buffer; padding keeps its old contents."""
    out = flat.copy()
    for (mat, eb, ec, off) in segments:
        out[off:off + ec] = np.ascontiguousarray(matrices[mat]).reshape(-1)[eb:eb + ec]
    return out


def layout_is_valid(flat_len: int, shapes: Sequence[Tuple[int, int]], segments, align: int,
                    num_shards: int, shard_len: int) -> bool:
    """Brute-force validity: every matrix element covered exactly once, flat ranges disjoint,
    aligned starts, every segment inside one shard."""
    if num_shards * shard_len != flat_len:
        return False
    cover = [np.zeros(m * n, dtype=np.int64) for (m, n) in shapes]
    used = np.zeros(flat_len, dtype=np.int64)
    for (mat, eb, ec, off) in segments:
        if not (0 <= mat < len(shapes)) or ec < 0 or eb < 0 or off < 0:
            return False
        if ec == 0:
            continue
        if eb + ec > cover[mat].size or off + ec > flat_len or off % align:
            return False
        if off // shard_len != (off + ec - 1) // shard_len:
            return False
        cover[mat][eb:eb + ec] += 1
        used[off:off + ec] += 1
    return all((c == 1).all() for c in cover) and (used <= 1).all()


# --------------------------------------------------------------------------- momentum (Section 2.3; Section 7.4 set-up: momentum 0.95, Nesterov)


def momentum_nesterov(G: np.ndarray, M: np.ndarray, mu: float, nesterov: bool = True) -> Tuple[np.ndarray, np.ndarray]:
    """M' = mu*M + G;  u = G + mu*M' (Nesterov) or u = M'.  M' is what the fp32 state stores."""
    G = np.asarray(G, dtype=np.float64)
    M = np.asarray(M, dtype=np.float64)
    M_new = mu * M + G
    u = G + mu * M_new if nesterov else M_new
    return M_new, u


# --------------------------------------------------------------------------- Newton-Schulz (Eq. 1, Section 6.6)


def _coeff(coeffs: Sequence[float], k: int) -> Tuple[float, float, float]:
    c = np.asarray(coeffs, dtype=np.float64).reshape(-1)
    if c.size == 3:
        return float(c[0]), float(c[1]), float(c[2])
    return float(c[3 * k]), float(c[3 * k + 1]), float(c[3 * k + 2])


def newton_schulz(U: np.ndarray, steps: int, coeffs: Sequence[float], eps: float = 1e-7, mode: str = "fp64",
                  trace: list | None = None) -> np.ndarray:
    """Orthogonalise U by `steps` iterations of Eq. 1, X_0 = U / (||U||_F + eps).

    Transpose-first rule (Section 6.6): when rows > cols the iteration runs on U^T so the
    Gram factor A = X X^T is the small square; the result is transposed back.

    The step of Eq. 1 is evaluated as the matrix polynomial it is: X_{k+1} = P_k X_k with
    P_k = a_k I + b_k A + c_k A^2, A = X_k X_k^T (three produced matrices per step: A, P, X).

    Rounding schedule in "bf16" mode ("cast then fold"): U is taken as given (already
    bf16-valued); the normaliser r = 1/(||U||_F + eps) is not applied to U but folded
    into the first step, A = r^2 (U U^T) and X_1 = r (P U), which equals Eq. 1 on
    X_0 = r U exactly in real arithmetic; each produced A, P, X is rounded once.
    `trace`, if given, receives (A, P, X) after every step (in the working orientation).
    """
    U = np.asarray(U, dtype=np.float64)
    rows, cols = U.shape
    tall = rows > cols
    X = U.T.copy() if tall else U.copy()
    if X.size == 0 or steps == 0:
        r = 1.0 / (np.sqrt(np.sum(X * X)) + eps) if X.size else 1.0
        X = _round(r * X, mode)
        return X.T.copy() if tall else X
    r = 1.0 / (np.sqrt(np.sum(X * X)) + eps)
    eye = np.eye(X.shape[0])
    for k in range(steps):
        a, b, c = _coeff(coeffs, k)
        if k == 0:
            A = _round((r * r) * np.matmul(X, X.T), mode)
            P = _round(a * eye + b * A + c * np.matmul(A, A), mode)
            X = _round(r * np.matmul(P, X), mode)
        else:
            A = _round(np.matmul(X, X.T), mode)
            P = _round(a * eye + b * A + c * np.matmul(A, A), mode)
            X = _round(np.matmul(P, X), mode)
        if trace is not None:
            trace.append((A.copy(), P.copy(), X.copy()))
    return X.T.copy() if tall else X


def ns_single_step(X: np.ndarray, a: float, b: float, c: float, mode: str = "fp64") -> np.ndarray:
    """One iteration of Eq. 1 on an already-normalised, wide-or-square X (teacher-forced checks)."""
    X = np.asarray(X, dtype=np.float64)
    A = _round(np.matmul(X, X.T), mode)
    P = _round(a * np.eye(X.shape[0]) + b * A + c * np.matmul(A, A), mode)
    return _round(np.matmul(P, X), mode)


# --------------------------------------------------------------------------- full step


def update_scale(rows: int, cols: int) -> float:
    """RMS-matching scale 0.2*sqrt(max(m, n)) (Section 2.3)."""
    return 0.2 * float(np.sqrt(max(rows, cols)))


def apply_update(W: np.ndarray, O: np.ndarray, lr: float, wd: float) -> np.ndarray:
    """W' = W (1 - lr*wd) - lr * 0.2 sqrt(max(m,n)) * O: decoupled decay acts on the old W (Section 6.3, Section 6.4 step 4)."""
    W = np.asarray(W, dtype=np.float64)
    rows, cols = W.shape
    return W * (1.0 - lr * wd) - lr * update_scale(rows, cols) * np.asarray(O, dtype=np.float64)


def muon_step(W: np.ndarray, G: np.ndarray, M: np.ndarray, lr: float, mu: float, wd: float, steps: int,
              coeffs: Sequence[float], eps: float = 1e-7, nesterov: bool = True, mode: str = "fp64"):
    """One Muon update of one matrix.  Returns (W', M', O) as float64 arrays.

    The optimizer state is fp32: M' and W' are rounded to float32 when stored, and in
    "bf16" mode the staged u is cast fp32 -> bf16 before orthogonalisation (the cast the
    fused gather performs on momentum shards, Section 6.4 step 1).
    """
    M_new, u = momentum_nesterov(G, M, mu, nesterov)
    M_store = M_new.astype(np.float32).astype(np.float64)
    if mode == "bf16":
        U = bf16_rne(u.astype(np.float32).astype(np.float64))
    else:
        U = u
    O = newton_schulz(U, steps, coeffs, eps, mode)
    W_new = apply_update(W, O, lr, wd).astype(np.float32).astype(np.float64)
    return W_new, M_store, O
