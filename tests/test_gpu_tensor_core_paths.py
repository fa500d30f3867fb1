"""GPU parity on batches of whole sequences at 512 to 8192 tokens, against the CPU oracle element
by element.  At these sizes the projections (compress, grad-project) and the fused
project-then-expand run on the tcgen05 kernels, while decompress takes the few-rows-per-SM
mma.sync kernel; the tcgen05 expansion and the large-batch mma.sync kernels are covered, with an
assertion of which kernel ran, in test_gpu_dispatch_coverage.py.  Also here: the prepared tables
EU = E U, PU = P U, the re-projection lists, guard bands and odd leading dimensions."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding, synth
from tests.harness import Codec, assert_close, f64, guards_intact, host64, padded, to_device

pytestmark = pytest.mark.gpu

# batch, seq_len, d, k, vocab
SHAPES = [
    (8, 128, 256, 40, 300),
    (32, 256, 1024, 40, 5000),
    (32, 64, 512, 16, 100),
    (256, 16, 384, 64, 100),
    (64, 48, 256, 33, 100),
    (8, 80, 128, 8, 50),
    (5, 200, 512, 40, 77),       # batch not a multiple of 8
    (3, 333, 256, 24, 77),       # sequence length not a multiple of 16
    (16, 64, 192, 40, 60),       # d not a multiple of 128
    (16, 64, 256, 72, 60),       # k > 64
    (12, 256, 2048, 128, 999),   # k = 128: two column groups of U; 24 tiles on 12 CTA pairs
    (17, 128, 1024, 96, 500),    # 17 tiles: the last pair splits its tile over d
    (1, 640, 512, 40, 200),      # 5 tiles on 3 pairs, one of them split
    (16, 128, 1024, 96, 500),    # 64 < k <= 128 on the expansion kernel, 8 x 16 tiles
    (8, 256, 512, 128, 300),
    (24, 64, 256, 72, 100),
    (8, 128, 64, 8, 40),         # d = 64: a single stage per tile, pairs cannot split it
    (9, 128, 128, 1, 40),        # k = 1, odd number of tiles
    (8, 128, 128, 16, 40),
]


def _inputs(batch, seq_len, d, k, vocab, seed):
    wl = synth.Workload("tc", d, k, vocab, batch, seq_len, synth.BF16)
    t = synth.codec_inputs(wl, seed=seed, noise_std=1e-3)
    return wl, t


@pytest.mark.parametrize("batch,seq_len,d,k,vocab", SHAPES)
@pytest.mark.parametrize("tables", ["EP", "E", "P", "none"])
def test_decompress_and_compress_on_sequence_batches(batch, seq_len, d, k, vocab, tables):
    wl, t = _inputs(batch, seq_len, d, k, vocab, seed=batch * 131 + seq_len + d + k)
    dt, n = wl.dtype, wl.n_tokens
    E0 = t["E"] if "E" in tables else None
    P0 = t["P"] if "P" in tables else None
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    U, E, P = f64(t["U"], dt), f64(E0, dt), f64(P0, dt)
    pos = oracle.token_positions(n, seq_len)

    Xh = codec.decompress(to_device(t["Z0"], dt), ids, seq_len=seq_len)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), U, E, t["ids"], P, pos)
    assert_close(host64(Xh, dt), Xo, dt, "decompress")

    X = to_device(t["X"], dt)
    Zo, _ = oracle.compress(f64(t["X"], dt), U, E, t["ids"], P, pos)
    assert_close(host64(codec.compress(X, ids, seq_len=seq_len), dt), Zo, dt, "compress")
    if tables != "none":
        codec.prepare_tables()
        assert_close(host64(codec.compress(X, ids, seq_len=seq_len), dt), Zo, dt, "compress, prepared tables")
        # one table only: the other term still comes from its rows
        for kw in (dict(embedding=False), dict(positions=False)):
            codec.prepare_tables(**kw)
            assert_close(host64(codec.compress(X, ids, seq_len=seq_len), dt), Zo, dt, f"compress, tables {kw}")
    assert codec.take_status() == 0


def test_prepared_tables_match_their_definition():
    for dt in (synth.F32, synth.BF16):
        wl = synth.Workload("tab", 384, 24, 211, 2, 96, dt)
        t = synth.codec_inputs(wl, seed=77)
        codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
        codec.prepare_tables()
        U, E, P = f64(t["U"], dt), f64(t["E"], dt), f64(t["P"], dt)
        for got, src in ((codec.EU, E), (codec.PU, P)):
            want = src @ U
            err = np.abs(got.double().cpu().numpy() - want).max() / np.abs(want).max()
            assert err < 2e-6, err


def test_prepared_tables_with_explicit_positions_and_bad_indices():
    """Explicit positions, a ragged token count, ids and positions out of range: the table path
    drops the same terms and raises the same status bits as the row path."""
    wl, t = _inputs(1, 1000, 512, 40, 90, seed=5)
    dt, n = wl.dtype, wl.n_tokens
    rng = np.random.default_rng(3)
    ids_np = t["ids"].copy()
    pos_np = rng.integers(0, wl.seq_len, n).astype(np.int32)
    ids_np[[3, 500]] = [-1, wl.vocab]
    pos_np[[7, 999]] = [wl.seq_len, -5]
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids, pos = torch.from_numpy(ids_np).cuda(), torch.from_numpy(pos_np).cuda()
    X = to_device(t["X"], dt)
    Zo, flags = oracle.compress(f64(t["X"], dt), f64(t["U"], dt), f64(t["E"], dt), ids_np,
                                f64(t["P"], dt), pos_np)
    Z_rows = codec.compress(X, ids, pos=pos)
    status_rows = codec.take_status()
    codec.prepare_tables()
    Z_tab = codec.compress(X, ids, pos=pos)
    status_tab = codec.take_status()
    assert_close(host64(Z_rows, dt), Zo, dt, "rows")
    assert_close(host64(Z_tab, dt), Zo, dt, "tables")
    assert status_rows == status_tab == (binding.SSN_DEV_BAD_ID | binding.SSN_DEV_BAD_POS) == flags


def test_prepare_tables_argument_errors():
    wl, t = _inputs(1, 64, 128, 8, 20, seed=1)
    dt = wl.dtype
    codec = Codec(dt, to_device(t["U"], dt))
    out = torch.empty((64, 8), dtype=torch.float32, device="cuda")
    fn = binding.raw("ssn_prepare_tables")
    assert fn(codec.c, out.data_ptr(), 8, None, 8, None) == binding.SSN_ERR_NULL      # no E in the codec
    codec2 = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt))
    assert fn(codec2.c, out.data_ptr(), 4, None, 8, None) == binding.SSN_ERR_SHAPE    # ldeu < k
    assert fn(codec2.c, None, 8, None, 8, None) == binding.SSN_OK                     # nothing to make


@pytest.mark.parametrize("rows,d,k", [(512, 256, 40), (1000, 512, 8), (2125, 1024, 64), (640, 384, 33),
                                      (3000, 2048, 16), (4096, 4096, 40), (3000, 2048, 128), (1024, 512, 96),
                                      (2000, 1024, 72)])
def test_project_then_expand_in_place_with_guard_bands(rows, d, k):
    """Weight re-projection (in place) and the projected gradient (out of place, with the
    coordinates) at sizes that take the fused tcgen05 kernel; nothing outside the rows moves."""
    dt = synth.BF16
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=rows + k), dt)
    W0 = synth.to_storage(np.random.default_rng(rows).standard_normal((rows, d)) * 0.05, dt)
    codec = Codec(dt, to_device(U0, dt))
    U, Wf = f64(U0, dt), f64(W0, dt)
    view, buf = padded(rows, d, d + 64, dt, fill=to_device(W0, dt))
    codec.weight_reproject([view], "right")
    assert_close(host64(view, dt), oracle.weight_reproject(Wf, U, "right"), dt, "reproject right")
    assert guards_intact(view, buf, dt)

    G = to_device(W0, dt)
    dZ, Gp = codec.grad_project(G, full=True)
    assert_close(host64(Gp, dt), oracle.grad_project_full(Wf, U), dt, "grad full")
    assert_close(host64(dZ, dt), oracle.grad_project_coeff(Wf, U), dt, "grad coeff")
    assert torch.equal(G, to_device(W0, dt))     # the input is not touched


def test_decompress_output_guard_bands_and_leading_dimensions():
    wl, t = _inputs(8, 64, 256, 40, 50, seed=9)
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    Zin, _ = padded(n, wl.k, wl.k + 24, dt, fill=to_device(t["Z0"], dt))
    out, buf = padded(n, wl.d, wl.d + 128, dt)
    codec.decompress(Zin, ids, seq_len=wl.seq_len, out=out)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), f64(t["U"], dt), f64(t["E"], dt), t["ids"],
                              f64(t["P"], dt), oracle.token_positions(n, wl.seq_len))
    assert_close(host64(out, dt), Xo, dt, "decompress into a padded view")
    assert guards_intact(out, buf, dt)
    assert codec.take_status() == 0


def test_reproject_rows_list_of_unequal_weights():
    """Several weights with different row counts in one call (one launch of the fused kernel),
    in place, against the oracle; then the shapes the fused kernel does not take."""
    dt, d, k = synth.BF16, 512, 40
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=3), dt)
    codec = Codec(dt, to_device(U0, dt))
    U = f64(U0, dt)
    rows = [640, 130, 1, 1024, 77, 256, 300, 128, 999, 64] + [96, 160, 33] * 9      # 37: more than one launch's worth
    W0s = [synth.to_storage(np.random.default_rng(r).standard_normal((r, d)) * 0.05, dt) for r in rows]
    views = [padded(r, d, d + 8 * (i % 3), dt, fill=to_device(w, dt)) for i, (r, w) in enumerate(zip(rows, W0s))]
    codec.weight_reproject_rows([v for v, _ in views])
    for (v, buf), w0 in zip(views, W0s):
        assert_close(host64(v, dt), oracle.weight_reproject(f64(w0, dt), U, "right"), dt, f"rows {v.shape[0]}")
        assert guards_intact(v, buf, dt)
    # fp32 and a rank above 64 take the general path, same results
    for dt2, k2 in ((synth.F32, 24), (synth.BF16, 72)):
        U2 = synth.to_storage(synth.subspace_basis(d, k2, seed=4), dt2)
        c2 = Codec(dt2, to_device(U2, dt2))
        Ws0 = [synth.to_storage(np.random.default_rng(r).standard_normal((r, d)) * 0.05, dt2) for r in (600, 50)]
        Ws = [to_device(w, dt2) for w in Ws0]
        c2.weight_reproject_rows(Ws)
        for w, w0 in zip(Ws, Ws0):
            assert_close(host64(w, dt2), oracle.weight_reproject(f64(w0, dt2), f64(U2, dt2), "right"), dt2, "general")


def test_reproject_list_left_side_unequal_columns():
    """LEFT side (W stored [d x m]): several weights of different widths in one call, in place,
    at sizes that take the fused kernel and at ones that take the general one."""
    dt, d, k = synth.BF16, 512, 40
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=5), dt)
    codec = Codec(dt, to_device(U0, dt))
    U = f64(U0, dt)
    cols = [512, 136, 1000, 8, 2048, 264, 128, 640, 72]
    W0s = [synth.to_storage(np.random.default_rng(c).standard_normal((d, c)) * 0.05, dt) for c in cols]
    views = [padded(d, c, c + 8 * (i % 3), dt, fill=to_device(w, dt)) for i, (c, w) in enumerate(zip(cols, W0s))]
    codec.weight_reproject_list([v for v, _ in views], "left")
    for (v, buf), w0 in zip(views, W0s):
        assert_close(host64(v, dt), oracle.weight_reproject(f64(w0, dt), U, "left"), dt, f"cols {v.shape[1]}")
        assert guards_intact(v, buf, dt)
    # odd widths and leading dimensions, fp32: the general kernels through the workspace
    for dt2, k2, widths in ((synth.BF16, 40, (333, 77)), (synth.F32, 24, (600, 50)), (synth.BF16, 136, (256,))):
        U2 = synth.to_storage(synth.subspace_basis(d, k2, seed=6), dt2)
        c2 = Codec(dt2, to_device(U2, dt2))
        Ws0 = [synth.to_storage(np.random.default_rng(c).standard_normal((d, c)) * 0.05, dt2) for c in widths]
        Ws = [to_device(w, dt2) for w in Ws0]
        c2.weight_reproject_list(Ws, "left")
        for w, w0 in zip(Ws, Ws0):
            assert_close(host64(w, dt2), oracle.weight_reproject(f64(w0, dt2), f64(U2, dt2), "left"), dt2, "general")
    # a weight that needs the workspace, without one
    odd = to_device(Ws0[0], dt2)
    with pytest.raises(binding.SsnError):
        binding.ssn_weight_reproject_list(c2.c, [odd.data_ptr()], [odd.shape[1]], [odd.shape[1]],
                                          binding.SIDES["left"])


@pytest.mark.parametrize("k", [16, 40, 64, 128])
def test_left_reprojection_of_the_8b_shapes(k):
    """The block's projections in the storage where the subspace is on the rows: out-proj
    [4096 x 4096] and down-proj [4096 x 14336], one call."""
    dt, d = synth.BF16, 4096
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=50 + k), dt)
    codec = Codec(dt, to_device(U0, dt))
    W0s = [synth.projection_weight(d, m, seed=9, dtype=dt, layer=i) for i, m in enumerate((4096, 14336))]
    Ws = [to_device(w, dt) for w in W0s]
    codec.weight_reproject_list(Ws, "left")
    for w, w0 in zip(Ws, W0s):
        assert_close(host64(w, dt), oracle.weight_reproject(f64(w0, dt), f64(U0, dt), "left"), dt, f"left k={k}")


def test_reproject_list_argument_errors():
    import ctypes
    dt, d, k = synth.BF16, 256, 8
    codec = Codec(dt, to_device(synth.to_storage(synth.subspace_basis(d, k, seed=3), dt), dt))
    W = torch.zeros((16, d), dtype=torch.bfloat16, device="cuda")
    fn = binding.raw("ssn_weight_reproject_list")
    ptrs, one = (ctypes.c_void_p * 1)(W.data_ptr()), ctypes.c_int64
    R = binding.SIDES["right"]
    assert fn(codec.c, ptrs, (one * 1)(16), (one * 1)(d), 1, R, None, 0, None) == binding.SSN_OK
    assert fn(codec.c, ptrs, (one * 1)(0), (one * 1)(d), 1, R, None, 0, None) == binding.SSN_ERR_SHAPE
    assert fn(codec.c, ptrs, (one * 1)(16), (one * 1)(d - 1), 1, R, None, 0, None) == binding.SSN_ERR_SHAPE
    assert fn(codec.c, None, (one * 1)(16), (one * 1)(d), 1, R, None, 0, None) == binding.SSN_ERR_NULL
    assert fn(codec.c, (ctypes.c_void_p * 1)(None), (one * 1)(16), (one * 1)(d), 1, R, None, 0, None) == binding.SSN_ERR_NULL
    assert fn(codec.c, ptrs, (one * 1)(16), (one * 1)(d), 0, R, None, 0, None) == binding.SSN_OK
    assert fn(codec.c, ptrs, (one * 1)(16), (one * 1)(d), -1, R, None, 0, None) == binding.SSN_ERR_SHAPE
    assert fn(codec.c, ptrs, (one * 1)(16), (one * 1)(d), 1, 7, None, 0, None) == binding.SSN_ERR_DTYPE
    L = binding.SIDES["left"]
    Wl = torch.zeros((d, 24), dtype=torch.bfloat16, device="cuda")
    pl = (ctypes.c_void_p * 1)(Wl.data_ptr())
    assert fn(codec.c, pl, (one * 1)(24), (one * 1)(23), 1, L, None, 0, None) == binding.SSN_ERR_SHAPE
    assert fn(codec.c, pl, (one * 1)(24), (one * 1)(24), 1, L, None, 0, None) == binding.SSN_ERR_WORKSPACE


def test_rank_that_is_not_a_multiple_of_8_with_padded_leading_dimensions():
    """k = 51 (the rank of the paper's 8B run): with U and Z stored at a leading dimension of 56
    every step takes the tensor-core kernels; results against the oracle, padding untouched."""
    from paper_2607_13332_b200.runner import padded_columns
    wl, t = _inputs(8, 256, 1024, 51, 300, seed=51)
    dt, n = wl.dtype, wl.n_tokens
    U = padded_columns(to_device(t["U"], dt))
    assert U.stride(0) == 56
    codec = Codec(dt, U, to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    Uf, Ef, Pf = f64(t["U"], dt), f64(t["E"], dt), f64(t["P"], dt)
    pos = oracle.token_positions(n, wl.seq_len)
    Zv, Zbuf = padded(n, wl.k, 56, dt)
    codec.compress(to_device(t["X"], dt), ids, seq_len=wl.seq_len, out=Zv)
    Zo, _ = oracle.compress(f64(t["X"], dt), Uf, Ef, t["ids"], Pf, pos)
    assert_close(host64(Zv, dt), Zo, dt, "compress")
    assert guards_intact(Zv, Zbuf, dt)
    Z0v, _ = padded(n, wl.k, 56, dt, fill=to_device(t["Z0"], dt))
    Xh = codec.decompress(Z0v, ids, seq_len=wl.seq_len)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), Uf, Ef, t["ids"], Pf, pos)
    assert_close(host64(Xh, dt), Xo, dt, "decompress")
    dZ, Gp = codec.grad_project(to_device(t["G"], dt), full=True)
    assert_close(host64(dZ, dt), oracle.grad_project_coeff(f64(t["G"], dt), Uf), dt, "grad coeff")
    assert_close(host64(Gp, dt), oracle.grad_project_full(f64(t["G"], dt), Uf), dt, "grad full")
    W0 = synth.projection_weight(640, wl.d, seed=2, dtype=dt)
    W = to_device(W0, dt)
    codec.weight_reproject_list([W], "right")
    assert_close(host64(W, dt), oracle.weight_reproject(f64(W0, dt), Uf, "right"), dt, "reproject")
    assert codec.take_status() == 0
