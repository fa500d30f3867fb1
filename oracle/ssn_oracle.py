"""Plain CPU oracle for the subspace-network (SSN) stage-boundary codec.

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this file.  It shares no code with the CUDA library and never calls it.

Every function is the paper's definition written out in float64 with numpy; the only library
primitive used as a step is a matrix product.  Nothing is blocked, fused or reordered.  Inputs
are float64 arrays holding the exact values of the stored (fp32 / bf16) tensors; outputs are
float64 and are not rounded.

Notation (paper Sec. 4.1, "Pipeline-Parallel Communication with Reparameterized SSNs"):
    X      [n, d]   hidden states, one row per token          (Eq. residual_stream)
    U      [d, k]   orthonormal basis U_k of the shared subspace, used exactly as stored
    E      [V, d]   fixed token embedding T_fixed; row ids[t] belongs to token t
    P      [S, d]   positional embedding PE; row pos[t] belongs to token t
    Z      [n, k]   the coordinates that cross the stage boundary   (Eq. ssn_compress)

Readings taken where the text is silent (they are listed with their reasons in the design
notes): the receiver adds E[ids] and P back after expanding with U^T; E and P are each
optional; a token whose id or position is out of range takes a zero row for that term and
raises a status bit instead of failing; the backward pass sends G U.

Pins (tests/test_oracle_pins.py): hand-worked example, one-hot basis special case, bit-exact
gather, isometry at k = d, exact round trip inside the subspace, adjoint and finite-difference
identities, projector identities, explicit d x d projector, element-by-element loops on tiny
shapes; for the reparameterized forms (Eq. reparam): the materialised weight W_p = Z U^T, its
membership of the subspace, loops, and the exact recovery of the factored embedding's coordinates
by compress; for compress_sum: linearity against a loop-written R U and the exact recovery of
summed coordinates; for the wire rows: IEEE-754 bit patterns typed by hand, the id word, the round trip
within half an fp32 ulp; for decompress_rowsumsq: the hand-worked example's rows squared by hand,
the closed form |Z|^2 + 2 <Z, s U> + |s|^2 for an orthonormal basis, loops, and the unit mean square
of the row it normalises.  No function here is left unpinned.
"""

from __future__ import annotations

from typing import Optional, Tuple

import numpy as np

STATUS_BAD_ID = 1
STATUS_BAD_POS = 2


def token_positions(n_tokens: int, seq_len: int) -> np.ndarray:
    """Position of token t when a [batch, seq_len] batch is flattened batch-major."""
    return np.arange(n_tokens, dtype=np.int64) % int(seq_len)


def shift_rows(n_tokens: int, d: int, E: Optional[np.ndarray], ids: Optional[np.ndarray],
               P: Optional[np.ndarray], pos: Optional[np.ndarray]) -> Tuple[np.ndarray, int]:
    """The per-token shift T_fixed[ids[t]] + PE[pos[t]] of Eq. ssn_compress, and a status word.

    A missing table contributes nothing.  An out-of-range index contributes a zero row and
    sets STATUS_BAD_ID / STATUS_BAD_POS.
    """
    shift = np.zeros((n_tokens, d), dtype=np.float64)
    status = 0
    if E is not None:
        ids = np.asarray(ids, dtype=np.int64)
        ok = (ids >= 0) & (ids < E.shape[0])
        if not ok.all():
            status |= STATUS_BAD_ID
        shift[ok] += np.asarray(E, dtype=np.float64)[ids[ok]]
    if P is not None:
        pos = np.asarray(pos, dtype=np.int64)
        ok = (pos >= 0) & (pos < P.shape[0])
        if not ok.all():
            status |= STATUS_BAD_POS
        shift[ok] += np.asarray(P, dtype=np.float64)[pos[ok]]
    return shift, status


def compress(X: np.ndarray, U: np.ndarray, E=None, ids=None, P=None, pos=None):
    """Eq. ssn_compress: Z = (X - PE - T_fixed) U_k.  Returns (Z [n, k], status)."""
    X = np.asarray(X, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    shift, status = shift_rows(X.shape[0], X.shape[1], E, ids, P, pos)
    return (X - shift) @ U, status


def compress_sum(X: np.ndarray, R: np.ndarray, U: np.ndarray, E=None, ids=None, P=None, pos=None):
    """Eq. ssn_compress applied to the hidden state of Eq. residual_stream written as residual stream
    plus the last block's output, X + R, the sum exact (float64).  Returns (Z [n, k], status)."""
    X = np.asarray(X, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    shift, status = shift_rows(X.shape[0], X.shape[1], E, ids, P, pos)
    return ((X + R) - shift) @ U, status


def decompress(Z: np.ndarray, U: np.ndarray, E=None, ids=None, P=None, pos=None):
    """Receiver side of Eq. ssn_compress: Xhat = Z U_k^T + PE + T_fixed.  Returns (Xhat, status)."""
    Z = np.asarray(Z, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    shift, status = shift_rows(Z.shape[0], U.shape[0], E, ids, P, pos)
    return Z @ U.T + shift, status


def decompress_rowsumsq(Z: np.ndarray, U: np.ndarray, E=None, ids=None, P=None, pos=None):
    """Receiver side fused with the row statistic of the receiving stage's first block: every
    block of the paper's models opens with an RMSNorm (model table of the experimental setup),
    whose only reduction is sum_i Xhat[t, i]^2 over the row that decompress has just produced
    (Sec. 4.1 puts decompress first on the receiving stage).  Returns (Xhat [n, d], rowsumsq [n],
    status); the squares are of the UNROUNDED reconstruction (the reading taken: the statistic is
    formed before the single rounding of Xhat to its storage type)."""
    Xhat, status = decompress(Z, U, E, ids, P, pos)
    return Xhat, (Xhat * Xhat).sum(axis=1), status


def grad_project_coeff(G: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Backward pass, "the same compression": the activation-gradient's coordinates dZ = G U_k."""
    return np.asarray(G, dtype=np.float64) @ np.asarray(U, dtype=np.float64)


def grad_project_full(G: np.ndarray, U: np.ndarray) -> np.ndarray:
    """The projected gradient itself, G U_k U_k^T (coordinates kept unrounded in between)."""
    U = np.asarray(U, dtype=np.float64)
    return grad_project_coeff(G, U) @ U.T


def weight_reproject(W: np.ndarray, U: np.ndarray, side: str) -> np.ndarray:
    """Original-SSN step after each optimizer update: put an output projection back in span(U).

    side = "right": W is [m, d] as in Eq. residual_stream (activations multiply it from the
    left), its rows must lie in the subspace:  W <- (W U) U^T.
    side = "left":  W is stored transposed, [d, m]:  W <- U (U^T W).
    """
    W = np.asarray(W, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    if side == "right":
        return (W @ U) @ U.T
    if side == "left":
        return U @ (U.T @ W)
    raise ValueError("side must be 'left' or 'right'")


def reparam_project(H: np.ndarray, Zw: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Eq. reparam: an output projection stored as its factor, W_p = Zw U_k^T.  The block's output
    Y = H W_p is formed as (H Zw) U_k^T, the k coordinates unrounded in between."""
    H = np.asarray(H, dtype=np.float64)
    return (H @ np.asarray(Zw, dtype=np.float64)) @ np.asarray(U, dtype=np.float64).T


def reparam_grad_factor(H: np.ndarray, dY: np.ndarray, U: np.ndarray) -> np.ndarray:
    """The chain rule quoted with Eq. reparam: dL/dZw = (dL/dW) U_k with dL/dW = H^T dY for Y = H W."""
    H = np.asarray(H, dtype=np.float64)
    return H.T @ (np.asarray(dY, dtype=np.float64) @ np.asarray(U, dtype=np.float64))


def head_embed(Elow: np.ndarray, U: np.ndarray, E=None, ids=None, P=None, pos=None):
    """Head-stage input with the factored trainable embedding T_S = Elow U_k^T (Sec. 4.1):
    X0[t] = T_fixed[ids[t]] + Elow[ids[t]] U_k^T + PE[pos[t]].  A token whose id is outside Elow
    contributes no trainable row (and, through decompress, no fixed row).  Returns (X0, status)."""
    Elow = np.asarray(Elow, dtype=np.float64)
    ids = np.asarray(ids, dtype=np.int64)
    ok = (ids >= 0) & (ids < Elow.shape[0])
    Z = np.zeros((ids.shape[0], Elow.shape[1]), dtype=np.float64)
    Z[ok] = Elow[ids[ok]]
    return decompress(Z, U, E, ids, P, pos)



def wire_rows(Z: np.ndarray, ids=None) -> np.ndarray:
    """Wire form of the boundary tensor (Sec. 3.5 sizes the boundary traffic in FP32): row t holds
    the k coordinates rounded to the nearest float32, as 32-bit words, followed (when ids is given)
    by the token id as an int32 word.  Returns an int32 array [n, k] or [n, k + 1]."""
    words = np.asarray(Z, dtype=np.float64).astype(np.float32).view(np.int32)
    if ids is None:
        return words.copy()
    return np.concatenate([words, np.asarray(ids, dtype=np.int32).reshape(-1, 1)], axis=1)


def wire_unpack(wire: np.ndarray, k: int, with_ids: bool):
    """Inverse of wire_rows: (coordinates as float64 [n, k], ids as int64 [n] or None)."""
    wire = np.ascontiguousarray(np.asarray(wire, dtype=np.int32))
    Z = wire[:, :k].copy().view(np.float32).astype(np.float64)
    return Z, (wire[:, k].astype(np.int64) if with_ids else None)
