"""GPU parity: every codec step through the C-ABI against the CPU oracle, element by element,
on the benchmark definition's workloads and on ragged / odd / degenerate shapes."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import synth
from tests.harness import (TOL, Codec, assert_close, f64, guards_intact, host64, padded, to_device,
                           to_host)

pytestmark = pytest.mark.gpu


def _run_all_steps(wl, t, sample=None, sides=("right",), wshape=None):
    """All four steps on one workload; oracle on all tokens or on the sampled ones."""
    dt = wl.dtype
    n = wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    X, G, Z0 = to_device(t["X"], dt), to_device(t["G"], dt), to_device(t["Z0"], dt)
    Z = codec.compress(X, ids, seq_len=wl.seq_len)
    Xh = codec.decompress(Z0, ids, seq_len=wl.seq_len)
    dZ, Gp = codec.grad_project(G, full=True)
    torch.cuda.synchronize()
    assert codec.take_status() == 0

    sel = np.arange(n) if sample is None else sample
    U, E, P = f64(t["U"], dt), f64(t["E"], dt), f64(t["P"], dt)
    pos = oracle.token_positions(n, wl.seq_len)[sel]
    idsel = t["ids"][sel]
    Zo, _ = oracle.compress(f64(t["X"][sel], dt), U, E, idsel, P, pos)
    Xo, _ = oracle.decompress(f64(t["Z0"][sel], dt), U, E, idsel, P, pos)
    Gsel = f64(t["G"][sel], dt)
    selt = torch.from_numpy(sel).cuda()
    errs = {
        "compress": assert_close(host64(Z[selt], dt), Zo, dt, f"{wl.name} compress"),
        "decompress": assert_close(host64(Xh[selt], dt), Xo, dt, f"{wl.name} decompress"),
        "grad coeff": assert_close(host64(dZ[selt], dt), oracle.grad_project_coeff(Gsel, U), dt,
                                   f"{wl.name} grad coeff"),
        "grad full": assert_close(host64(Gp[selt], dt), oracle.grad_project_full(Gsel, U), dt,
                                  f"{wl.name} grad full"),
    }
    return codec, errs


def test_config0_tiny_fp32_all_steps():
    wl = synth.TINY
    for noise in (0.0, 1e-3):
        t = synth.codec_inputs(wl, seed=0x5EED, noise_std=noise)
        codec, _ = _run_all_steps(wl, t)
        for side, shape in (("right", (512, 512)), ("left", (512, 512))):
            W0 = synth.projection_weight(*shape, seed=7, dtype=wl.dtype)
            W = to_device(W0, wl.dtype)
            codec.weight_reproject([W], side)
            expect = oracle.weight_reproject(f64(W0, wl.dtype), f64(t["U"], wl.dtype), side)
            assert_close(host64(W, wl.dtype), expect, wl.dtype, f"tiny reproject {side}")


def test_config1_mid_bf16_all_steps():
    wl = synth.MID
    t = synth.codec_inputs(wl, seed=0x5EED + 16)
    codec, _ = _run_all_steps(wl, t)
    # the MLP down-projection stored [d x 4d]: the subspace is on the left
    W0 = synth.projection_weight(2048, 8192, seed=8, dtype=wl.dtype)
    W = to_device(W0, wl.dtype)
    codec.weight_reproject([W], "left")
    expect = oracle.weight_reproject(f64(W0, wl.dtype), f64(t["U"], wl.dtype), "left")
    assert_close(host64(W, wl.dtype), expect, wl.dtype, "mid reproject left")


def test_config2_stage8b_full_size_sampled():
    """The 8B-class boundary at full size (65536 tokens, Zipf ids), oracle on sampled tokens:
    first and last 256 tokens plus 2048 seeded random ones."""
    wl = synth.STAGE_8B
    t = synth.codec_inputs(wl, seed=0x5EED + 32)
    n = wl.n_tokens
    rng = np.random.default_rng(1)
    sample = np.unique(np.concatenate([np.arange(256), np.arange(n - 256, n),
                                       rng.integers(0, n, 2048)]))
    _run_all_steps(wl, t, sample=sample)


@pytest.mark.parametrize("k", synth.REPROJECT_RANKS)
def test_config3_reprojection_sweep(k):
    d, dt = 4096, synth.BF16
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=40 + k), dt)
    codec = Codec(dt, to_device(U0, dt))
    U = f64(U0, dt)
    for name, (rows, cols) in synth.REPROJECT_SHAPES_8B.items():
        sides = ("right", "left") if rows == cols else ("right",)
        for side in sides:
            W0s = [synth.projection_weight(rows, cols, seed=9, dtype=dt, layer=l) for l in range(2)]
            Ws = [to_device(w, dt) for w in W0s]
            codec.weight_reproject(Ws, side)
            for w0, w in zip(W0s, Ws):
                expect = oracle.weight_reproject(f64(w0, dt), U, side)
                assert_close(host64(w, dt), expect, dt, f"{name} {side} k={k}")


# ---------------------------------------------------------------------------------------
# ragged, odd and degenerate shapes
# ---------------------------------------------------------------------------------------
EDGE_SHAPES = [
    # n, d, k, vocab, seq_len, dtype
    (1, 64, 1, 5, 3, synth.F32),
    (37, 96, 5, 17, 8, synth.F32),
    (300, 512, 8, 100, 64, synth.F32),
    (1, 256, 8, 9, 4, synth.BF16),
    (129, 256, 51, 33, 7, synth.BF16),        # rank of the paper's 8B run: not a multiple of 8
    (1000, 1024, 40, 500, 33, synth.BF16),    # several tiles and a ragged tail
    (257, 200, 5, 20, 10, synth.BF16),        # d not a multiple of 32
    (515, 2048, 128, 64, 100, synth.BF16),
    (77, 128, 128, 10, 11, synth.BF16),       # k == d
]


@pytest.mark.parametrize("n,d,k,vocab,seq_len,dt", EDGE_SHAPES)
@pytest.mark.parametrize("tables", ["EP", "E", "P", "none"])
def test_edge_shapes(n, d, k, vocab, seq_len, dt, tables):
    wl = synth.Workload("edge", d, k, vocab, 1, n, dt)
    t = synth.codec_inputs(wl, seed=n + d + k, noise_std=1e-3)
    rng = np.random.default_rng(n)
    pos_np = rng.integers(0, seq_len, n).astype(np.int32)        # explicit positions
    P0 = synth.to_storage(synth.sinusoidal_positions(seq_len, d), dt)
    E0 = t["E"] if "E" in tables else None
    P0 = P0 if "P" in tables else None
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    pos = torch.from_numpy(pos_np).cuda()
    U, E, P = f64(t["U"], dt), f64(E0, dt), f64(P0, dt)

    X = to_device(t["X"], dt)
    Z = codec.compress(X, ids, pos=pos)
    Zo, _ = oracle.compress(f64(t["X"], dt), U, E, t["ids"], P, pos_np)
    assert_close(host64(Z, dt), Zo, dt, "compress")

    Xh = codec.decompress(to_device(t["Z0"], dt), ids, pos=pos)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), U, E, t["ids"], P, pos_np)
    assert_close(host64(Xh, dt), Xo, dt, "decompress")

    if tables == "none":
        G = to_device(t["G"], dt)
        dZ, Gp = codec.grad_project(G, full=True)
        assert_close(host64(dZ, dt), oracle.grad_project_coeff(f64(t["G"], dt), U), dt, "grad coeff")
        assert_close(host64(Gp, dt), oracle.grad_project_full(f64(t["G"], dt), U), dt, "grad full")
        only_full = codec.grad_project(G, full=True, coeff=False)
        assert torch.equal(only_full, Gp)
        for side in ("right", "left"):
            W0 = t["X"] if side == "right" else np.ascontiguousarray(t["X"].T)
            W = to_device(W0, dt)
            codec.weight_reproject([W], side)
            assert_close(host64(W, dt), oracle.weight_reproject(f64(W0, dt), U, side), dt,
                         f"reproject {side}")
    assert codec.take_status() == 0


@pytest.mark.parametrize("dt", [synth.F32, synth.BF16])
def test_leading_dimensions_unaligned_views_and_guard_bands(dt):
    n, d, k, vocab, seq_len = 203, 320, 24, 50, 16
    wl = synth.Workload("ld", d, k, vocab, 1, n, dt)
    t = synth.codec_inputs(wl, seed=99, noise_std=1e-3)
    # every matrix lives in a wider buffer at an offset of one element: odd leading
    # dimensions, pointers that are not 16-byte aligned
    Uv, _ = padded(d, k, k + 3, dt, to_device(t["U"], dt))
    Ev, _ = padded(vocab, d, d + 5, dt, to_device(t["E"], dt))
    Pv, _ = padded(seq_len, d, d + 1, dt, to_device(synth.to_storage(
        synth.sinusoidal_positions(seq_len, d), dt), dt))
    Xv, _ = padded(n, d, d + 7, dt, to_device(t["X"], dt))
    Z0v, _ = padded(n, k, k + 1, dt, to_device(t["Z0"], dt))
    codec = Codec(dt, Uv, Ev, Pv)
    ids = torch.from_numpy(t["ids"]).cuda()
    U, E, P = host64(Uv, dt), host64(Ev, dt), host64(Pv, dt)
    pos = oracle.token_positions(n, seq_len)

    Zv, Zbuf = padded(n, k, k + 9, dt)
    codec.compress(Xv, ids, seq_len=seq_len, out=Zv)
    assert guards_intact(Zv, Zbuf, dt)
    assert_close(host64(Zv, dt), oracle.compress(f64(t["X"], dt), U, E, t["ids"], P, pos)[0], dt, "compress")

    Xhv, Xbuf = padded(n, d, d + 3, dt)
    codec.decompress(Z0v, ids, seq_len=seq_len, out=Xhv)
    assert guards_intact(Xhv, Xbuf, dt)
    assert_close(host64(Xhv, dt), oracle.decompress(f64(t["Z0"], dt), U, E, t["ids"], P, pos)[0], dt,
                 "decompress")

    dZv, dZbuf = padded(n, k, k + 2, dt)
    Gpv, Gpbuf = padded(n, d, d + 11, dt)
    codec.grad_project(Xv, full=True, out=dZv, out_full=Gpv)
    assert guards_intact(dZv, dZbuf, dt) and guards_intact(Gpv, Gpbuf, dt)
    assert_close(host64(dZv, dt), oracle.grad_project_coeff(f64(t["X"], dt), U), dt, "grad coeff")
    assert_close(host64(Gpv, dt), oracle.grad_project_full(f64(t["X"], dt), U), dt, "grad full")

    for side in ("right", "left"):
        W0 = t["X"] if side == "right" else np.ascontiguousarray(t["X"].T)
        Wv, Wbuf = padded(W0.shape[0], W0.shape[1], W0.shape[1] + 5, dt, to_device(W0, dt))
        codec.weight_reproject([Wv], side)
        assert guards_intact(Wv, Wbuf, dt)
        assert_close(host64(Wv, dt), oracle.weight_reproject(f64(W0, dt), U, side), dt, f"reproject {side}")


@pytest.mark.parametrize("dt", [synth.F32, synth.BF16])
@pytest.mark.parametrize("d,k", [(256, 8), (4096, 40)])
def test_gathered_rows_are_bit_exact(dt, d, k):
    """Z = 0 and no positional table: the receiver must hand back E[ids] bit for bit (a stored
    -0 may come back as +0); and X = E[ids] must compress to exactly zero."""
    wl = synth.Workload("gather", d, k, 700, 3, 111, dt, "zipf")
    t = synth.codec_inputs(wl, seed=5, with_positions=False)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    Zero = torch.zeros((wl.n_tokens, k), dtype=codec.U.dtype, device="cuda")
    Xh = to_host(codec.decompress(Zero, ids), dt)
    rows = t["E"][t["ids"]]
    same_bits = Xh.view(np.uint32 if dt == synth.F32 else np.uint16) == \
        rows.view(np.uint32 if dt == synth.F32 else np.uint16)
    both_zero = (f64(Xh, dt) == 0) & (f64(rows, dt) == 0)
    assert bool(np.all(same_bits | both_zero))
    Z = codec.compress(to_device(rows, dt), ids)
    assert bool((Z == 0).all())
    assert codec.take_status() == 0


def test_one_hot_basis_is_a_bit_exact_subtraction_fp32():
    dt = synth.F32
    n, d, k, vocab = 130, 128, 16, 40
    wl = synth.Workload("onehot", d, k, vocab, 1, n, dt)
    t = synth.codec_inputs(wl, seed=6, noise_std=0.1, with_positions=False)
    U = np.eye(d, dtype=np.float32)[:, :k].copy()
    codec = Codec(dt, to_device(U, dt), to_device(t["E"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    Z = to_host(codec.compress(to_device(t["X"], dt), ids), dt)
    expect = (t["X"] - t["E"][t["ids"]])[:, :k]          # one correctly rounded fp32 subtraction
    np.testing.assert_array_equal(Z, expect)


def test_out_of_range_ids_and_positions_set_status_and_zero_the_row():
    dt = synth.BF16
    n, d, k, vocab, seq_len = 64, 256, 8, 30, 8
    wl = synth.Workload("bad", d, k, vocab, 1, n, dt)
    t = synth.codec_inputs(wl, seed=7)
    P0 = synth.to_storage(synth.sinusoidal_positions(seq_len, d), dt)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(P0, dt))
    ids_np = t["ids"].copy()
    pos_np = (np.arange(n) % seq_len).astype(np.int32)
    U, E, P = f64(t["U"], dt), f64(t["E"], dt), f64(P0, dt)
    for bad_ids, bad_pos, bits in (([3], [], 1), ([], [5, 60], 2), ([0, 63], [17], 3)):
        i2, p2 = ids_np.copy(), pos_np.copy()
        i2[bad_ids] = vocab + 5
        if bad_ids:
            i2[bad_ids[-1]] = -2
        p2[bad_pos] = seq_len
        X = to_device(t["X"], dt)
        Z = codec.compress(X, torch.from_numpy(i2).cuda(), pos=torch.from_numpy(p2).cuda())
        torch.cuda.synchronize()
        assert codec.take_status() == bits
        Zo, st = oracle.compress(f64(t["X"], dt), U, E, i2, P, p2)
        assert st == bits
        assert_close(host64(Z, dt), Zo, dt, "compress with bad indices")
        Xh = codec.decompress(to_device(t["Z0"], dt), torch.from_numpy(i2).cuda(),
                              pos=torch.from_numpy(p2).cuda())
        assert codec.take_status() == bits
        assert_close(host64(Xh, dt), oracle.decompress(f64(t["Z0"], dt), U, E, i2, P, p2)[0], dt,
                     "decompress with bad indices")


def test_round_trip_on_device_is_lossless_inside_the_subspace():
    wl = synth.MID.scaled(batch=2)
    t = synth.codec_inputs(wl, seed=8)
    dt = wl.dtype
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    X = to_device(t["X"], dt)
    Z = codec.compress(X, ids, seq_len=wl.seq_len)
    Xh = codec.decompress(Z, ids, seq_len=wl.seq_len)
    assert_close(host64(Z, dt), f64(t["Z0"], dt), dt, "coordinates recovered", tol=2e-2)
    assert_close(host64(Xh, dt), f64(t["X"], dt), dt, "activation recovered", tol=2e-2)
