"""Pins for the CPU oracle: every check here is fixed by the paper's equations or by plain
mathematics, never by the oracle's own formula retyped with the same library call."""

import os

import numpy as np
import pytest

from oracle import ssn_oracle as oracle
from oracle.metrics import max_rel_err
from paper_2607_13332_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------
# A hand-worked example of Eq. ssn_compress (d=4, k=2, three tokens).
#   u1 = (1,1,1,1)/2, u2 = (1,-1,1,-1)/2 are orthonormal.
#   E[0] = (1,0,0,0), E[1] = (0,2,0,0);  P[0] = 0, P[1] = (0,0,1,1);  ids = 1,0,1; pos = 0,1,0.
#   token 0: X=(1,2,3,4):  X-E[1]-P[0] = (1,0,3,4)   -> (8/2, 0/2)           = (4, 0)
#   token 1: X=(2,0,1,-1): X-E[0]-P[1] = (1,0,0,-2)  -> ((1-2)/2, (1+2)/2)   = (-0.5, 1.5)
#   token 2: X=(0,2,0,0):  X-E[1]-P[0] = 0           -> (0, 0)
#   back:  4 u1 = (2,2,2,2), + E[1] = (2,4,2,2)
#          -0.5 u1 + 1.5 u2 = (0.5,-1,0.5,-1), + E[0] + P[1] = (1.5,-1,1.5,0)
# ---------------------------------------------------------------------------------------
U4 = np.array([[.5, .5], [.5, -.5], [.5, .5], [.5, -.5]])
E4 = np.array([[1., 0, 0, 0], [0, 2., 0, 0]])
P4 = np.array([[0., 0, 0, 0], [0, 0, 1., 1.]])
IDS4 = np.array([1, 0, 1])
POS4 = np.array([0, 1, 0])
X4 = np.array([[1., 2, 3, 4], [2, 0, 1, -1], [0, 2, 0, 0]])
Z4 = np.array([[4., 0], [-0.5, 1.5], [0, 0]])
XHAT4 = np.array([[2., 4, 2, 2], [1.5, -1, 1.5, 0], [0, 2, 0, 0]])


def test_hand_worked_compress():
    Z, status = oracle.compress(X4, U4, E4, IDS4, P4, POS4)
    assert status == 0
    np.testing.assert_allclose(Z, Z4, rtol=0, atol=1e-15)


def test_hand_worked_decompress():
    Xh, status = oracle.decompress(Z4, U4, E4, IDS4, P4, POS4)
    assert status == 0
    np.testing.assert_allclose(Xh, XHAT4, rtol=0, atol=1e-15)


def test_hand_worked_grad_and_reproject():
    R = np.array([[1., 0, 3, 4], [1, 0, 0, -2]])          # two rows worked above
    T = np.array([[4., 0], [-0.5, 1.5]])
    RP = np.array([[2., 2, 2, 2], [0.5, -1, 0.5, -1]])
    np.testing.assert_allclose(oracle.grad_project_coeff(R, U4), T, atol=1e-15)
    np.testing.assert_allclose(oracle.grad_project_full(R, U4), RP, atol=1e-15)
    np.testing.assert_allclose(oracle.weight_reproject(R, U4, "right"), RP, atol=1e-15)
    np.testing.assert_allclose(oracle.weight_reproject(R.T.copy(), U4, "left"), RP.T, atol=1e-15)


def test_hand_worked_row_sum_of_squares():
    # rows of XHAT4 squared by hand: 4+16+4+4, 2.25+1+2.25+0, 0+4+0+0
    Xh, ss, status = oracle.decompress_rowsumsq(Z4, U4, E4, IDS4, P4, POS4)
    assert status == 0
    np.testing.assert_allclose(Xh, XHAT4, rtol=0, atol=1e-15)
    np.testing.assert_allclose(ss, [28.0, 5.5, 4.0], rtol=0, atol=1e-14)


def test_row_sum_of_squares_closed_form_loops_and_normalisation():
    """For orthonormal U and shift s = E[id] + P[pos]:  |Z U^T + s|^2 = |Z|^2 + 2 <Z, s U> + |s|^2,
    each term written with explicit loops; without a shift the statistic is |Z|^2 (isometry); and
    dividing the row by sqrt(rowsumsq / d) leaves a unit mean square (what RMSNorm does with it)."""
    rng = np.random.default_rng(12)
    n, d, k, vocab, seq = 7, 12, 3, 5, 4
    U = synth.subspace_basis(d, k, seed=12)
    E, P = rng.standard_normal((vocab, d)), rng.standard_normal((seq, d))
    Z = rng.standard_normal((n, k))
    ids, pos = rng.integers(0, vocab, n), rng.integers(0, seq, n)
    Xh, ss, _ = oracle.decompress_rowsumsq(Z, U, E, ids, P, pos)
    for t in range(n):
        shift = [E[ids[t]][i] + P[pos[t]][i] for i in range(d)]
        zz = sum(Z[t][j] ** 2 for j in range(k))
        cross = sum(Z[t][j] * sum(shift[i] * U[i][j] for i in range(d)) for j in range(k))
        assert abs(ss[t] - (zz + 2 * cross + sum(v * v for v in shift))) < 1e-11
        row = [sum(Z[t][j] * U[i][j] for j in range(k)) + shift[i] for i in range(d)]     # the definition, by loops
        assert abs(ss[t] - sum(v * v for v in row)) < 1e-11
        normed = Xh[t] / np.sqrt(ss[t] / d)
        assert abs(float(np.mean(normed ** 2)) - 1.0) < 1e-12
    _, ss0, _ = oracle.decompress_rowsumsq(Z, U)
    np.testing.assert_allclose(ss0, [sum(Z[t][j] ** 2 for j in range(k)) for t in range(n)], rtol=1e-12)


def test_positions_default_is_t_mod_seq_len():
    np.testing.assert_array_equal(oracle.token_positions(7, 3), [0, 1, 2, 0, 1, 2, 0])
    np.testing.assert_array_equal(oracle.token_positions(3, 2), POS4)


# ---------------------------------------------------------------------------------------
# Element-by-element loops on small shapes (no matrix product, different index order).
# ---------------------------------------------------------------------------------------
def _small_problem(seed, n=7, d=12, k=5, V=9, S=4):
    rng = np.random.default_rng(seed)
    U = np.linalg.qr(rng.standard_normal((d, k)))[0]
    E = rng.standard_normal((V, d))
    P = rng.standard_normal((S, d))
    ids = rng.integers(0, V, n)
    pos = rng.integers(0, S, n)
    X = rng.standard_normal((n, d))
    Z = rng.standard_normal((n, k))
    return U, E, P, ids, pos, X, Z


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_loops_compress_decompress(seed):
    U, E, P, ids, pos, X, Z = _small_problem(seed)
    n, d = X.shape
    k = U.shape[1]
    Zl = np.zeros((n, k))
    Xl = np.zeros((n, d))
    for t in range(n):
        for j in range(k):
            acc = 0.0
            for i in range(d):
                acc += (X[t, i] - P[pos[t], i] - E[ids[t], i]) * U[i, j]
            Zl[t, j] = acc
        for i in range(d):
            acc = 0.0
            for j in range(k):
                acc += U[i, j] * Z[t, j]
            Xl[t, i] = acc + P[pos[t], i] + E[ids[t], i]
    np.testing.assert_allclose(oracle.compress(X, U, E, ids, P, pos)[0], Zl, atol=1e-13)
    np.testing.assert_allclose(oracle.decompress(Z, U, E, ids, P, pos)[0], Xl, atol=1e-13)
    # each table is optional and independent of the other
    np.testing.assert_allclose(oracle.compress(X, U, E, ids)[0] - oracle.compress(X, U)[0],
                               -(E[ids] @ U), atol=1e-13)
    np.testing.assert_allclose(oracle.compress(X, U, None, None, P, pos)[0] - oracle.compress(X, U)[0],
                               -(P[pos] @ U), atol=1e-13)


@pytest.mark.parametrize("seed", [3, 4])
def test_loops_grad_and_reproject(seed):
    U, _, _, _, _, G, _ = _small_problem(seed, n=6, d=10, k=3)
    n, d = G.shape
    k = U.shape[1]
    dZ = np.zeros((n, k))
    for t in range(n):
        for j in range(k):
            dZ[t, j] = sum(G[t, i] * U[i, j] for i in range(d))
    np.testing.assert_allclose(oracle.grad_project_coeff(G, U), dZ, atol=1e-13)
    Gp = np.zeros((n, d))
    for t in range(n):
        for i in range(d):
            Gp[t, i] = sum(dZ[t, j] * U[i, j] for j in range(k))
    np.testing.assert_allclose(oracle.grad_project_full(G, U), Gp, atol=1e-13)
    # right: rows of W are projected; left: columns of W are projected
    np.testing.assert_allclose(oracle.weight_reproject(G, U, "right"), Gp, atol=1e-13)
    W = np.random.default_rng(seed).standard_normal((d, 4))
    Wl = np.zeros_like(W)
    for c in range(4):
        t = [sum(U[i, j] * W[i, c] for i in range(d)) for j in range(k)]
        for i in range(d):
            Wl[i, c] = sum(U[i, j] * t[j] for j in range(k))
    np.testing.assert_allclose(oracle.weight_reproject(W, U, "left"), Wl, atol=1e-13)


# ---------------------------------------------------------------------------------------
# Special cases that reduce to something that needs no arithmetic at all.
# ---------------------------------------------------------------------------------------
def test_one_hot_basis_selects_columns():
    rng = np.random.default_rng(5)
    n, d, k, V, S = 9, 16, 4, 11, 3
    U = np.eye(d)[:, :k]
    E, P = rng.standard_normal((V, d)), rng.standard_normal((S, d))
    ids, pos = rng.integers(0, V, n), oracle.token_positions(n, S)
    X, Z = rng.standard_normal((n, d)), rng.standard_normal((n, k))
    got, _ = oracle.compress(X, U, E, ids, P, pos)
    np.testing.assert_allclose(got, (X - E[ids] - P[pos])[:, :k], rtol=0, atol=1e-15)
    # with one table only there is a single subtraction per element: exact
    got, _ = oracle.compress(X, U, E, ids)
    for t in range(n):
        for j in range(k):
            assert got[t, j] == X[t, j] - E[ids[t], j]
    Xh, _ = oracle.decompress(Z, U, E, ids, P, pos)
    np.testing.assert_allclose(Xh[:, :k], Z + E[ids][:, :k] + P[pos][:, :k], atol=1e-15)
    np.testing.assert_array_equal(Xh[:, k:], (E[ids] + P[pos])[:, k:])


def test_gather_is_exact():
    wl = synth.Workload("g", d=64, k=4, vocab=50, batch=2, seq_len=8, dtype=synth.BF16)
    t = synth.codec_inputs(wl, seed=11)
    E = synth.to_f64(t["E"], wl.dtype)
    U = synth.to_f64(t["U"], wl.dtype)
    Xh, status = oracle.decompress(np.zeros((wl.n_tokens, wl.k)), U, E, t["ids"])
    assert status == 0
    for tok in range(wl.n_tokens):
        np.testing.assert_array_equal(Xh[tok], E[t["ids"][tok]])
    Z, _ = oracle.compress(E[t["ids"]], U, E, t["ids"])
    np.testing.assert_array_equal(Z, np.zeros_like(Z))


def test_isometry_when_k_equals_d():
    rng = np.random.default_rng(6)
    d = 24
    U = np.linalg.qr(rng.standard_normal((d, d)))[0]
    E, P = rng.standard_normal((5, d)), rng.standard_normal((4, d))
    ids, pos = rng.integers(0, 5, 10), rng.integers(0, 4, 10)
    X = rng.standard_normal((10, d))
    Z, _ = oracle.compress(X, U, E, ids, P, pos)
    np.testing.assert_allclose(np.linalg.norm(Z, axis=1),
                               np.linalg.norm(X - E[ids] - P[pos], axis=1), rtol=1e-13)
    Xh, _ = oracle.decompress(Z, U, E, ids, P, pos)
    np.testing.assert_allclose(Xh, X, atol=1e-12)    # a full basis loses nothing


def test_out_of_range_indices_zero_row_and_status():
    U, E, P, ids, pos, X, Z = _small_problem(7)
    ids = ids.copy(); pos = pos.copy()
    ids[2] = E.shape[0]; ids[3] = -1; pos[4] = P.shape[0]
    Zc, status = oracle.compress(X, U, E, ids, P, pos)
    assert status == (oracle.STATUS_BAD_ID | oracle.STATUS_BAD_POS)
    np.testing.assert_allclose(Zc[2], (X[2] - P[pos[2]]) @ U, atol=1e-13)
    np.testing.assert_allclose(Zc[3], (X[3] - P[pos[3]]) @ U, atol=1e-13)
    np.testing.assert_allclose(Zc[4], (X[4] - E[ids[4]]) @ U, atol=1e-13)
    Xh, status = oracle.decompress(Z, U, E, ids, None, None)
    assert status == oracle.STATUS_BAD_ID
    np.testing.assert_allclose(Xh[2], U @ Z[2], atol=1e-13)


# ---------------------------------------------------------------------------------------
# Invariants the paper states: orthonormal basis, lossless inside the subspace.
# ---------------------------------------------------------------------------------------
def test_basis_is_orthonormal():
    for d, k in [(512, 8), (2048, 32), (4096, 40)]:
        U = synth.subspace_basis(d, k, seed=1)
        assert np.max(np.abs(U.T @ U - np.eye(k))) <= 1e-13
        Ub = synth.to_f64(synth.to_storage(U, synth.BF16), synth.BF16)
        assert np.max(np.abs(Ub.T @ Ub - np.eye(k))) <= 2.0 ** -7


def test_round_trip_inside_subspace_is_lossless():
    # X built here by explicit loops, not by the oracle and not by the generator
    rng = np.random.default_rng(8)
    n, d, k, V, S = 10, 32, 6, 13, 5
    U = synth.subspace_basis(d, k, seed=3)
    E, P = rng.standard_normal((V, d)), rng.standard_normal((S, d))
    ids, pos = rng.integers(0, V, n), oracle.token_positions(n, S)
    Z0 = rng.standard_normal((n, k))
    X = np.zeros((n, d))
    for t in range(n):
        for i in range(d):
            X[t, i] = E[ids[t], i] + P[pos[t], i] + sum(Z0[t, j] * U[i, j] for j in range(k))
    Z, _ = oracle.compress(X, U, E, ids, P, pos)
    np.testing.assert_allclose(Z, Z0, atol=1e-12)
    Xh, _ = oracle.decompress(Z, U, E, ids, P, pos)
    np.testing.assert_allclose(Xh, X, atol=1e-12)


def test_off_subspace_noise_is_what_is_lost():
    rng = np.random.default_rng(9)
    n, d, k = 12, 40, 7
    U = synth.subspace_basis(d, k, seed=4)
    E = rng.standard_normal((6, d))
    ids = rng.integers(0, 6, n)
    Z0 = rng.standard_normal((n, k))
    N = 1e-3 * rng.standard_normal((n, d))
    X = E[ids] + Z0 @ U.T + N
    Z, _ = oracle.compress(X, U, E, ids)
    np.testing.assert_allclose(Z - Z0, N @ U, atol=1e-13)
    Xh, _ = oracle.decompress(Z, U, E, ids)
    lost = N - (N @ U) @ U.T
    np.testing.assert_allclose(X - Xh, lost, atol=1e-13)
    # what the receiver rebuilds minus the shift has nothing outside span(U)
    R = Xh - E[ids]
    np.testing.assert_allclose(R - (R @ U) @ U.T, 0, atol=1e-13)


def test_generated_workload_round_trip():
    # the generator's X lies in the shifted subspace up to fp32 storage rounding
    wl = synth.Workload("t", d=128, k=8, vocab=64, batch=2, seq_len=16, dtype=synth.F32)
    t = synth.codec_inputs(wl, seed=21)
    f = lambda name: synth.to_f64(t[name], wl.dtype)
    pos = oracle.token_positions(wl.n_tokens, wl.seq_len)
    Z, _ = oracle.compress(f("X"), f("U"), f("E"), t["ids"], f("P"), pos)
    assert max_rel_err(Z, f("Z0")) < 5e-6


def test_compress_is_linear_in_the_residual():
    rng = np.random.default_rng(10)
    U = synth.subspace_basis(20, 3, seed=5)
    A, B = rng.standard_normal((4, 20)), rng.standard_normal((4, 20))
    lhs = oracle.compress(2.5 * A - 0.75 * B, U)[0]
    rhs = 2.5 * oracle.compress(A, U)[0] - 0.75 * oracle.compress(B, U)[0]
    np.testing.assert_allclose(lhs, rhs, atol=1e-13)


# ---------------------------------------------------------------------------------------
# Backward pass: the projection is the transpose of the receiver's expansion (chain rule).
# ---------------------------------------------------------------------------------------
def test_grad_project_is_adjoint_of_expansion():
    rng = np.random.default_rng(12)
    n, d, k = 9, 30, 5
    U = synth.subspace_basis(d, k, seed=6)
    G, Zt = rng.standard_normal((n, d)), rng.standard_normal((n, k))
    lhs = np.sum(oracle.grad_project_coeff(G, U) * Zt)
    rhs = np.sum(G * oracle.decompress(Zt, U)[0])
    assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs))


def test_grad_project_matches_finite_differences():
    rng = np.random.default_rng(13)
    n, d, k = 3, 14, 4
    U = synth.subspace_basis(d, k, seed=7)
    E, ids = rng.standard_normal((5, d)), rng.integers(0, 5, n)
    T = rng.standard_normal((n, d))
    Z = rng.standard_normal((n, k))
    loss = lambda z: 0.5 * np.sum((oracle.decompress(z, U, E, ids)[0] - T) ** 2)
    upstream = oracle.decompress(Z, U, E, ids)[0] - T          # dL/dXhat
    analytic = oracle.grad_project_coeff(upstream, U)
    h = 1e-6
    for t in range(n):
        for j in range(k):
            zp, zm = Z.copy(), Z.copy()
            zp[t, j] += h; zm[t, j] -= h
            numeric = (loss(zp) - loss(zm)) / (2 * h)
            assert abs(numeric - analytic[t, j]) < 1e-7


def test_grad_full_is_idempotent_and_fixes_the_subspace():
    rng = np.random.default_rng(14)
    U = synth.subspace_basis(36, 6, seed=8)
    G = rng.standard_normal((8, 36))
    once = oracle.grad_project_full(G, U)
    np.testing.assert_allclose(oracle.grad_project_full(once, U), once, atol=1e-13)
    inside = rng.standard_normal((8, 6)) @ U.T
    np.testing.assert_allclose(oracle.grad_project_full(inside, U), inside, atol=1e-13)


# ---------------------------------------------------------------------------------------
# Weight re-projection: an orthogonal projector applied to rows (right) or columns (left).
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("side", ["left", "right"])
def test_reproject_projector_identities(side):
    rng = np.random.default_rng(15)
    d, k, m = 48, 7, 20
    U = synth.subspace_basis(d, k, seed=9)
    W = rng.standard_normal((d, m) if side == "left" else (m, d))
    PW = oracle.weight_reproject(W, U, side)
    np.testing.assert_allclose(oracle.weight_reproject(PW, U, side), PW, atol=1e-13)
    resid = W - PW
    if side == "left":
        np.testing.assert_allclose(U.T @ resid, 0, atol=1e-13)
        fixed = U @ rng.standard_normal((k, m))
    else:
        np.testing.assert_allclose(resid @ U, 0, atol=1e-13)
        fixed = rng.standard_normal((m, k)) @ U.T      # the paper's W = Z U^T factorisation
    np.testing.assert_allclose(oracle.weight_reproject(fixed, U, side), fixed, atol=1e-13)
    assert np.linalg.norm(PW) <= np.linalg.norm(W) * (1 + 1e-14)
    # explicit d x d projector
    Pi = np.zeros((d, d))
    for j in range(k):
        Pi += np.outer(U[:, j], U[:, j])
    expect = Pi @ W if side == "left" else W @ Pi
    np.testing.assert_allclose(PW, expect, atol=1e-13)


def test_reproject_left_is_right_on_the_transpose():
    rng = np.random.default_rng(16)
    U = synth.subspace_basis(24, 5, seed=10)
    W = rng.standard_normal((24, 9))
    np.testing.assert_allclose(oracle.weight_reproject(W, U, "left"),
                               oracle.weight_reproject(W.T.copy(), U, "right").T, atol=1e-14)


# ---------------------------------------------------------------------------------------
# Sizes the paper prints.
# ---------------------------------------------------------------------------------------
def test_paper_boundary_sizes():
    vals = {}
    with open(os.path.join(GOLDEN, "paper_sizes.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                name, value = line.split()
                vals[name] = int(value)
    bits = vals["tokens_8b"] * vals["d_8b"] * vals["bits_per_value"]
    assert bits == 671_088_640 and round(bits / 1e6) == vals["boundary_mbit_8b"]
    assert round(vals["d_8b"] / vals["rank_8b"]) == vals["compression_8b"]
    # the coordinates of one 8B microbatch in FP32
    Z, _ = oracle.compress(np.zeros((vals["tokens_8b"], 8)), np.zeros((8, 1)))
    assert Z.shape == (vals["tokens_8b"], 1)
    assert vals["tokens_8b"] * vals["rank_8b"] * 4 == 835_584
    assert abs(vals["d_1b"] / vals["rank_1b"] - 51.2) < 1e-12


# ---------------------------------------------------------------------------------------
# reparameterized forms (Eq. reparam)
# ---------------------------------------------------------------------------------------
def test_reparam_project_is_the_materialised_weight():
    """Y = (H Z) U^T must be H W_p with W_p = Z U^T written out, W_p must lie in the subspace
    (re-projecting it changes nothing), and a hand-sized case is checked with loops."""
    rng = np.random.default_rng(11)
    n, m, d, k = 7, 13, 24, 5
    U = synth.subspace_basis(d, k, seed=1)
    H, Zw = rng.standard_normal((n, m)), rng.standard_normal((m, k))
    W = np.zeros((m, d))
    for r in range(m):
        for c in range(d):
            W[r, c] = sum(Zw[r, j] * U[c, j] for j in range(k))
    Y = oracle.reparam_project(H, Zw, U)
    expect = np.zeros((n, d))
    for t in range(n):
        for c in range(d):
            expect[t, c] = sum(H[t, r] * W[r, c] for r in range(m))
    assert np.abs(Y - expect).max() < 1e-12
    assert np.abs(oracle.weight_reproject(W, U, "right") - W).max() < 1e-12
    # the coordinates the next boundary would send are H Zw: compressing Y gives them back
    Z, _ = oracle.compress(Y, U)
    assert np.abs(Z - H @ Zw).max() < 1e-12


def test_reparam_factor_gradient_is_the_projected_weight_gradient():
    """Chain rule quoted with Eq. reparam: dL/dZ = (dL/dW) U_k, checked by finite differences of
    L = <Y, R> through reparam_project."""
    rng = np.random.default_rng(12)
    n, m, d, k = 5, 6, 16, 3
    U = synth.subspace_basis(d, k, seed=2)
    H, Zw, R = rng.standard_normal((n, m)), rng.standard_normal((m, k)), rng.standard_normal((n, d))
    grad_W = H.T @ R                                   # dL/dW for Y = H W
    analytic = grad_W @ U
    assert np.abs(oracle.reparam_grad_factor(H, R, U) - analytic).max() < 1e-12
    eps = 1e-6
    for r, j in ((0, 0), (3, 2), (5, 1)):
        Zp, Zm = Zw.copy(), Zw.copy()
        Zp[r, j] += eps
        Zm[r, j] -= eps
        fd = (np.sum(oracle.reparam_project(H, Zp, U) * R) - np.sum(oracle.reparam_project(H, Zm, U) * R)) / (2 * eps)
        assert abs(fd - analytic[r, j]) < 1e-7


def test_head_embed_is_gather_of_the_materialised_table_and_is_recovered_by_compress():
    rng = np.random.default_rng(13)
    V, d, k, n, S = 17, 32, 4, 40, 8
    U = synth.subspace_basis(d, k, seed=3)
    Elow, E, P = rng.standard_normal((V, k)), rng.standard_normal((V, d)), rng.standard_normal((S, d))
    ids = rng.integers(0, V, n)
    pos = oracle.token_positions(n, S)
    X0, status = oracle.head_embed(Elow, U, E, ids, P, pos)
    T_S = Elow @ U.T                                   # the trainable table written out
    expect = np.stack([E[ids[t]] + T_S[ids[t]] + P[pos[t]] for t in range(n)])
    assert status == 0 and np.abs(X0 - expect).max() < 1e-12
    Z, _ = oracle.compress(X0, U, E, ids, P, pos)      # "entirely lossless" (Sec. 4.1)
    assert np.abs(Z - Elow[ids]).max() < 1e-12
    bad = ids.copy()
    bad[2] = V
    X1, status = oracle.head_embed(Elow, U, E, bad, P, pos)
    assert status == oracle.STATUS_BAD_ID and np.abs(X1[2] - P[pos[2]]).max() == 0.0



# ---- wire rows -------------------------------------------------------------------------------
def test_wire_rows_bit_patterns():
    """IEEE-754 single patterns typed by hand: 1.0, -2.5, 0.1 (rounds to 0x3DCCCCCD), 0; the id word."""
    Z = np.array([[1.0, -2.5], [0.1, 0.0]])
    w = oracle.wire_rows(Z, ids=[7, 128255])
    assert w.dtype == np.int32 and w.shape == (2, 3)
    as_u32 = w.view(np.uint32)
    assert as_u32[0, 0] == 0x3F800000 and as_u32[0, 1] == 0xC0200000
    assert as_u32[1, 0] == 0x3DCCCCCD and as_u32[1, 1] == 0
    assert w[0, 2] == 7 and w[1, 2] == 128255
    assert oracle.wire_rows(Z).shape == (2, 2)


def test_wire_round_trip_half_ulp():
    rng = np.random.default_rng(5)
    Z = rng.standard_normal((37, 11)) * np.exp(rng.uniform(-20, 20, size=(37, 11)))
    ids = rng.integers(0, 2 ** 31 - 1, size=37)
    back, ids_back = oracle.wire_unpack(oracle.wire_rows(Z, ids), 11, True)
    assert np.array_equal(ids_back, ids)
    assert np.all(np.abs(back - Z) <= np.abs(Z) * 2.0 ** -24)
    # values that are float32 already travel unchanged
    Z32 = Z.astype(np.float32).astype(np.float64)
    assert np.array_equal(oracle.wire_unpack(oracle.wire_rows(Z32), 11, False)[0], Z32)


# ---- compress fused with the residual add ------------------------------------------------------
def test_compress_sum_linearity_and_recovery():
    rng = np.random.default_rng(11)
    n, d, k, V, S = 9, 12, 4, 7, 5
    U, _ = np.linalg.qr(rng.standard_normal((d, k)))
    E, P = rng.standard_normal((V, d)), rng.standard_normal((S, d))
    ids, pos = rng.integers(0, V, n), np.arange(n) % S
    X, R = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    Zs, status = oracle.compress_sum(X, R, U, E, ids, P, pos)
    assert status == 0
    RU = np.zeros((n, k))                                  # R U with loops
    for t_ in range(n):
        for j in range(k):
            for i in range(d):
                RU[t_, j] += R[t_, i] * U[i, j]
    np.testing.assert_allclose(Zs - oracle.compress(X, U, E, ids, P, pos)[0], RU, atol=1e-12)
    # a hidden state split in two parts inside the shifted subspace gives the summed coordinates back
    Za, Zb = rng.standard_normal((n, k)), rng.standard_normal((n, k))
    Xa = Za @ U.T + E[ids] + P[pos]
    Rb = Zb @ U.T
    np.testing.assert_allclose(oracle.compress_sum(Xa, Rb, U, E, ids, P, pos)[0], Za + Zb, atol=1e-12)
    # swapping the addends changes nothing; a zero residual is plain compress
    np.testing.assert_allclose(oracle.compress_sum(R, X, U, E, ids, P, pos)[0], Zs, atol=1e-12)
    np.testing.assert_array_equal(oracle.compress_sum(X, np.zeros_like(X), U, E, ids, P, pos)[0],
                                  oracle.compress(X, U, E, ids, P, pos)[0])


# ---- data-parallel ops: AsyncSPARTA round, stage-wise clipping ---------------------------------
def test_sparta_round_from_steps_is_the_plain_mean():
    """Eq. sparta: after a round every replica's buf[I] is the mean over replicas; assembled here
    from the steps of Algorithm 3 with equal weights, and a weighted round with a weight-0 sender."""
    from oracle import dp_oracle as dp
    rng = np.random.default_rng(2)
    n, R = 2003, 4
    bufs = [rng.standard_normal(n) for _ in range(R)]
    lo, hi = dp.sparta_segment(n, 20, 7)
    assert (lo, hi) == (640, 768)                            # floor(701.05) and floor(801.2) down to 64s
    for weights in ([1.0] * R, [3.0, 0.0, 1.0, 2.0]):
        chunks = [dp.sparta_snapshot(b, lo, hi) for b in bufs]
        acc = np.zeros(hi - lo)
        for c, w in zip(chunks, weights):
            acc = dp.sparta_accumulate(acc, c, w)
        mean, deltas = dp.sparta_deltas(acc, sum(weights), chunks)
        expect = sum(w * b[lo:hi] for w, b in zip(weights, bufs)) / sum(weights)
        np.testing.assert_allclose(mean, expect, atol=1e-13)
        for b, dlt in zip(bufs, deltas):
            after = dp.sparta_add_delta(b, lo, hi, dlt)
            np.testing.assert_allclose(after[lo:hi], expect, atol=1e-13)      # the group average
            assert np.array_equal(after[:lo], b[:lo]) and np.array_equal(after[hi:], b[hi:])
    # the weight-0 sender (index 1) changed nothing for the others: same mean without it
    rest = [0, 2, 3]
    np.testing.assert_allclose(expect, sum([3.0, 1.0, 2.0][i] * bufs[j][lo:hi] for i, j in enumerate(rest)) / 6.0,
                               atol=1e-13)


def test_sparta_segments_tile_a_cycle():
    from oracle import dp_oracle as dp
    for n in (0, 1, 19, 20, 1000, 8_030_261_248 // 7):
        covered = 0
        for r in range(20):
            lo, hi = dp.sparta_segment(n, 20, r)
            assert lo == covered and hi >= lo and lo % 64 == 0
            assert abs(lo - n * r / 20) < 64                 # within one alignment unit of the even split
            covered = hi
        assert covered == n
        assert dp.sparta_segment(n, 20, 27) == dp.sparta_segment(n, 20, 7)


def test_delta_rule_keeps_local_progress():
    """Eq. delta_rule: theta + (avg - snap); the local update theta - snap survives on top of the
    average, and with no local progress (theta == snap) the result is the average itself."""
    from oracle import dp_oracle as dp
    rng = np.random.default_rng(3)
    n, lo, hi = 50, 10, 30
    theta, snap_full = rng.standard_normal(n), rng.standard_normal(n)
    avg = rng.standard_normal(hi - lo)
    snap = snap_full[lo:hi]
    out = dp.sparta_apply_round(theta, lo, hi, avg, snap)
    np.testing.assert_allclose(out[lo:hi] - avg, theta[lo:hi] - snap, atol=1e-13)
    assert np.array_equal(out[:lo], theta[:lo]) and np.array_equal(out[hi:], theta[hi:])
    np.testing.assert_allclose(dp.sparta_apply_round(snap_full, lo, hi, avg, snap)[lo:hi], avg, atol=1e-13)
    np.testing.assert_allclose(dp.sparta_apply_round(theta, lo, hi, avg, snap, lam=0.0), theta, atol=0)


def test_stage_clip_thresholds_printed_in_the_paper():
    """Table 1 lists 0.3779 / 0.3779 / 0.7558 for head / body / tail of the 7-stage run."""
    from oracle import dp_oracle as dp
    golden = [float(v) for v in open(os.path.join(os.path.dirname(__file__), "golden",
                                                  "stage_clip_thresholds.txt")).read().split()[-3:]]
    assert golden == [0.3779, 0.3779, 0.7558]
    assert abs(dp.stage_clip_threshold(7, False) - golden[0]) < 1e-4
    assert abs(dp.stage_clip_threshold(7, True) - golden[2]) < 2e-4
    assert dp.stage_clip_threshold(1, False) == 1.0          # one stage: the usual global threshold of 1
    # S stages at their thresholds stay inside the unit budget: sum of squares = 1
    assert abs(sum(dp.stage_clip_threshold(7, False) ** 2 for _ in range(7)) - 1.0) < 1e-12


def test_stage_clip_norm_and_identity():
    from oracle import dp_oracle as dp
    rng = np.random.default_rng(4)
    grads = [rng.standard_normal((5, 7)), rng.standard_normal(11), rng.standard_normal((2, 3, 4))]
    norm = np.sqrt(sum(float((g ** 2).sum()) for g in grads))
    c = 0.3779
    clipped, got_norm, coef = dp.stage_clip(grads, c)
    assert abs(got_norm - norm) < 1e-12 and coef < 1
    new_norm = np.sqrt(sum(float((g ** 2).sum()) for g in clipped))
    assert abs(new_norm - c) < 1e-5                          # min(norm, c) up to the 1e-6 guard
    for g, h in zip(grads, clipped):                         # the direction is unchanged
        np.testing.assert_allclose(h * norm, g * new_norm, atol=1e-12)
    small = [g * (0.1 / norm) for g in grads]
    same, _, coef1 = dp.stage_clip(small, c)
    assert coef1 == 1.0 and all(np.array_equal(a, b) for a, b in zip(same, small))
