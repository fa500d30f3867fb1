"""GPU parity of the wire-row entry points (k fp32 coordinates + the token id per token; Sec. 3.5
sizes the boundary traffic in FP32) against the oracle: compress_wire, grad_project_wire and
decompress_wire on the tensor-core and the general kernels."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding, synth
from tests.harness import Codec, assert_close, f64, host64, to_device

pytestmark = pytest.mark.gpu

WIRE_TOL = 1e-5          # fp32 coordinates, whatever the storage dtype of X
GUARD = 0x5A5A5A5A

# batch, seq_len, d, k, vocab, dtype
CASES = [
    (8, 128, 512, 40, 300, synth.BF16),      # tcgen05 projection; decompress with rank 80 (two groups)
    (16, 128, 1024, 24, 500, synth.BF16),    # decompress with rank 48 (one group)
    (8, 256, 256, 64, 100, synth.BF16),      # rank 128, the largest the split form takes
    (9, 128, 384, 33, 200, synth.BF16),      # odd rank: scalar stores, padded rank 40
    (8, 128, 256, 72, 100, synth.BF16),      # 2 * 72 > 128: decompress on the general kernel
    (3, 50, 128, 5, 40, synth.BF16),         # few tokens
    (5, 100, 136, 8, 60, synth.BF16),        # d not a multiple of 32: general kernels throughout
    (2, 64, 128, 8, 30, synth.F32),
]


def wire_buffer(n, words, ldw):
    buf = torch.full((n + 2, ldw), GUARD, dtype=torch.int32, device="cuda")
    return buf[1:n + 1], buf


def wire_guards_intact(buf, n, words):
    ok = bool((buf[0] == GUARD).all()) and bool((buf[n + 1] == GUARD).all())
    return ok and bool((buf[1:n + 1, words:] == GUARD).all())


@pytest.mark.parametrize("batch,seq_len,d,k,vocab,dt", CASES)
@pytest.mark.parametrize("with_ids", [True, False])
def test_compress_wire(batch, seq_len, d, k, vocab, dt, with_ids):
    wl = synth.Workload("wire", d, k, vocab, batch, seq_len, dt)
    t = synth.codec_inputs(wl, seed=batch + d + k, noise_std=0.05)
    n = wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    words = k + (1 if with_ids else 0)
    for ldw in (words, (words + 3) // 4 * 4 + 4):          # packed rows, then a 16-byte aligned pitch
        view, buf = wire_buffer(n, words, ldw)
        codec.compress_wire(to_device(t["X"], dt), ids, seq_len=seq_len, with_ids=with_ids, out=view)
        assert codec.take_status() == 0
        expect, _ = oracle.compress(f64(t["X"], dt), f64(t["U"], dt), f64(t["E"], dt), t["ids"], f64(t["P"], dt),
                                    oracle.token_positions(n, seq_len))
        got, got_ids = oracle.wire_unpack(view[:, :words].cpu().numpy(), k, with_ids)
        assert_close(got, expect, dt, "wire coordinates", tol=WIRE_TOL)
        if with_ids:
            assert np.array_equal(got_ids, t["ids"])
        assert wire_guards_intact(buf, n, words)
    # the prepared tables give the same rows within the same bound
    codec.prepare_tables()
    w2 = codec.compress_wire(to_device(t["X"], dt), ids, seq_len=seq_len, with_ids=with_ids)
    assert_close(oracle.wire_unpack(w2.cpu().numpy(), k, with_ids)[0], expect, dt, "wire coordinates, tables",
                 tol=WIRE_TOL)


@pytest.mark.parametrize("batch,seq_len,d,k,vocab,dt", CASES)
def test_grad_project_wire(batch, seq_len, d, k, vocab, dt):
    wl = synth.Workload("wire", d, k, vocab, batch, seq_len, dt)
    t = synth.codec_inputs(wl, seed=batch + d)
    codec = Codec(dt, to_device(t["U"], dt))
    dZ = codec.grad_project_wire(to_device(t["G"], dt))
    assert dZ.dtype == torch.float32
    expect = oracle.grad_project_coeff(f64(t["G"], dt), f64(t["U"], dt))
    assert_close(dZ.cpu().numpy().astype(np.float64), expect, dt, "dZ wire", tol=WIRE_TOL)


@pytest.mark.parametrize("batch,seq_len,d,k,vocab,dt", CASES)
@pytest.mark.parametrize("with_ids", [True, False])
def test_decompress_wire(batch, seq_len, d, k, vocab, dt, with_ids):
    wl = synth.Workload("wire", d, k, vocab, batch, seq_len, dt)
    t = synth.codec_inputs(wl, seed=batch + k)
    n = wl.n_tokens
    rng = np.random.default_rng(d + k)
    Z = rng.standard_normal((n, k))                       # full fp32 mantissas, not bf16 values
    ids_np = t["ids"].copy()
    ids_np[2] = vocab + 5                                 # one id outside the table
    pos = oracle.token_positions(n, seq_len)
    wire_np = oracle.wire_rows(Z, ids_np if with_ids else None)
    Zw, _ = oracle.wire_unpack(wire_np, k, with_ids)
    expect, status = oracle.decompress(Zw, f64(t["U"], dt), f64(t["E"], dt), ids_np, f64(t["P"], dt), pos)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    wire = torch.from_numpy(wire_np).cuda()
    ids = None if with_ids else torch.from_numpy(ids_np).cuda()
    for use_ws in (True, False):                          # split form on the tensor cores / general kernel
        Xh = codec.decompress_wire(wire, ids, seq_len=seq_len, with_ids=with_ids, use_workspace=use_ws)
        assert_close(host64(Xh, dt), expect, dt, f"decompress from wire rows (workspace {use_ws})")
        assert codec.take_status() == status == binding.SSN_DEV_BAD_ID
    assert torch.equal(wire, torch.from_numpy(wire_np).cuda())


def test_wire_round_trip_keeps_fp32_coordinates():
    """compress_wire then decompress_wire inside the shifted subspace: the error of X^ is the
    rounding of X and X^ alone (the coordinates are not rounded to bf16 in between)."""
    dt = synth.BF16
    wl = synth.Workload("wire", 512, 40, 300, 8, 128, dt)
    t = synth.codec_inputs(wl, seed=3)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    wire = codec.compress_wire(to_device(t["X"], dt), ids, seq_len=128, with_ids=True)
    Xh = codec.decompress_wire(wire, seq_len=128, with_ids=True)
    assert_close(host64(Xh, dt), f64(t["X"], dt), dt, "wire round trip")


def test_wire_argument_errors():
    dt = synth.BF16
    wl = synth.Workload("wire", 128, 8, 50, 2, 64, dt)
    t = synth.codec_inputs(wl, seed=1)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    X = to_device(t["X"], dt)
    ids = torch.from_numpy(t["ids"]).cuda()
    n = wl.n_tokens
    wire = codec.wire_buffer(n, True)
    with pytest.raises(binding.SsnError) as e:             # the id word does not fit
        binding.ssn_compress_wire(codec.c, X.data_ptr(), 128, ids.data_ptr(), 0, n, 64, wire.data_ptr(), 8, True)
    assert e.value.status == binding.SSN_ERR_SHAPE
    codec_no_e = Codec(dt, to_device(t["U"], dt))
    with pytest.raises(binding.SsnError) as e:             # ids to pack, none given
        binding.ssn_compress_wire(codec_no_e.c, X.data_ptr(), 128, 0, 0, n, 64, wire.data_ptr(), 9, True)
    assert e.value.status == binding.SSN_ERR_NULL
    Xh = torch.empty_like(X)
    with pytest.raises(binding.SsnError) as e:             # ids inside the rows need a workspace
        binding.ssn_decompress_wire(codec.c, wire.data_ptr(), 9, True, 0, 0, n, 64, Xh.data_ptr(), 128, 0, 0)
    assert e.value.status == binding.SSN_ERR_WORKSPACE
    assert binding.ssn_decompress_wire_workspace_bytes(codec.c, n, True) >= n * 4 + n * 16 * 2 + 128 * 16 * 2
    assert binding.ssn_decompress_wire_workspace_bytes(codec.c, n, False) > 0
    binding.ssn_compress_wire(codec.c, X.data_ptr(), 128, ids.data_ptr(), 0, 0, 64, 0, 9, True)   # empty batch


# batch, seq_len, d, k, vocab, dtype
SUM_CASES = [
    (8, 128, 512, 40, 300, synth.BF16),
    (9, 128, 1024, 64, 500, synth.BF16),     # odd tile count: a pair splits its last tile between X and R
    (75, 128, 256, 16, 100, synth.BF16),     # more tiles than CTA pairs
    (8, 128, 256, 96, 100, synth.BF16),      # two coordinate groups
    (8, 128, 64, 8, 50, synth.BF16),         # one stage per matrix
    (3, 50, 128, 5, 40, synth.BF16),         # few tokens: general kernel
    (2, 64, 128, 8, 30, synth.F32),
]


@pytest.mark.parametrize("batch,seq_len,d,k,vocab,dt", SUM_CASES)
def test_compress_sum(batch, seq_len, d, k, vocab, dt):
    """Z = (X + R - E - P) U on a codec with prepared tables (tensor cores), with gathered rows
    (general kernel) and without E and P, in the three output forms."""
    wl = synth.Workload("sum", d, k, vocab, batch, seq_len, dt)
    t = synth.codec_inputs(wl, seed=batch + d + k, noise_std=0.05)
    n = wl.n_tokens
    rng = np.random.default_rng(batch + k)
    R0 = synth.to_storage(rng.standard_normal((n, d)) * 0.3, dt)
    X, R = to_device(t["X"], dt), to_device(R0, dt)
    ids = torch.from_numpy(t["ids"]).cuda()
    pos = oracle.token_positions(n, seq_len)
    Uf, Ef, Pf = f64(t["U"], dt), f64(t["E"], dt), f64(t["P"], dt)
    expect, _ = oracle.compress_sum(f64(t["X"], dt), f64(R0, dt), Uf, Ef, t["ids"], Pf, pos)
    rows = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    tables = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    tables.prepare_tables()
    for name, codec in (("gathered rows", rows), ("prepared tables", tables)):
        Z = codec.compress_sum(X, R, ids, seq_len=seq_len)
        assert_close(host64(Z, dt), expect, dt, f"compress_sum, {name}")
        w = codec.compress_sum(X, R, ids, seq_len=seq_len, wire=True, with_ids=True)
        got, got_ids = oracle.wire_unpack(w.cpu().numpy(), k, True)
        assert_close(got, expect, dt, f"compress_sum wire rows, {name}", tol=WIRE_TOL)
        assert np.array_equal(got_ids, t["ids"])
        assert codec.take_status() == 0
    bare = Codec(dt, to_device(t["U"], dt))
    w = bare.compress_sum(X, R, wire=True)
    assert_close(oracle.wire_unpack(w.cpu().numpy(), k, False)[0],
                 oracle.compress_sum(f64(t["X"], dt), f64(R0, dt), Uf)[0], dt, "compress_sum, no tables", tol=WIRE_TOL)
    assert torch.equal(X, to_device(t["X"], dt)) and torch.equal(R, to_device(R0, dt))


def test_compress_sum_argument_errors():
    dt = synth.BF16
    wl = synth.Workload("sum", 128, 8, 50, 2, 64, dt)
    t = synth.codec_inputs(wl, seed=1)
    codec = Codec(dt, to_device(t["U"], dt))
    X = to_device(t["X"], dt)
    Z = torch.empty((wl.n_tokens, 8), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.SsnError) as e:
        binding.ssn_compress_sum(codec.c, X.data_ptr(), 128, 0, 128, 0, 0, wl.n_tokens, 64, Z.data_ptr(), 8)
    assert e.value.status == binding.SSN_ERR_NULL
    with pytest.raises(binding.SsnError) as e:
        binding.ssn_compress_sum(codec.c, X.data_ptr(), 128, X.data_ptr(), 64, 0, 0, wl.n_tokens, 64, Z.data_ptr(), 8)
    assert e.value.status == binding.SSN_ERR_SHAPE
    with pytest.raises(binding.SsnError) as e:
        binding.ssn_compress_sum(codec.c, X.data_ptr(), 128, X.data_ptr(), 128, 0, 0, wl.n_tokens, 64, Z.data_ptr(), 8, 7)
    assert e.value.status == binding.SSN_ERR_DTYPE
