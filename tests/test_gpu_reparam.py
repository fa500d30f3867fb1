"""GPU parity of the reparameterized-SSN entry points (Eq. reparam): the output projection from its
factor, Y = (H Zw) U^T, and the head-stage input with the factored embedding, against the oracle."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding, synth
from tests.harness import Codec, assert_close, f64, guards_intact, host64, padded, to_device

pytestmark = pytest.mark.gpu

# n, m, d, k, dtype: tensor-core shapes (n >= 512, m % 64 == 0, d % 128 == 0) and general ones
CASES = [
    (2048, 1024, 512, 40, synth.BF16),
    (1000, 3584, 1024, 40, synth.BF16),      # ragged token count, m != d
    (640, 256, 384, 33, synth.BF16),
    (4096, 14336, 4096, 40, synth.BF16),     # the 8B block's MLP down-projection
    (768, 512, 256, 128, synth.BF16),        # two 64-coordinate groups
    (600, 512, 512, 96, synth.BF16),
    (100, 96, 64, 5, synth.BF16),            # few tokens, odd shapes: general kernels
    (515, 200, 136, 8, synth.BF16),
    (300, 128, 128, 8, synth.F32),
]


@pytest.mark.parametrize("n,m,d,k,dt", CASES)
def test_reparam_project(n, m, d, k, dt):
    rng = np.random.default_rng(n + m + d + k)
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=n + k), dt)
    H0 = synth.to_storage(rng.standard_normal((n, m)) * 0.5, dt)
    Zw0 = synth.to_storage(rng.standard_normal((m, k)) / np.sqrt(m), dt)
    codec = Codec(dt, to_device(U0, dt))
    H, Zw = to_device(H0, dt), to_device(Zw0, dt)
    out, buf = padded(n, d, d + 64, dt)
    coords, cbuf = padded(n, k, -(-k // 8) * 8 + 8, dt)
    codec.reparam_project(H, Zw, out=out, coords=coords)
    expect = oracle.reparam_project(f64(H0, dt), f64(Zw0, dt), f64(U0, dt))
    assert_close(host64(out, dt), expect, dt, "Y = (H Zw) U^T")
    assert_close(host64(coords, dt), f64(H0, dt) @ f64(Zw0, dt), dt, "coordinates H Zw")
    assert guards_intact(out, buf, dt) and guards_intact(coords, cbuf, dt)
    assert torch.equal(H, to_device(H0, dt))
    # without the coordinates output
    Y2 = codec.reparam_project(H, Zw)
    assert_close(host64(Y2, dt), expect, dt, "Y, no coordinates")


@pytest.mark.parametrize("batch,seq_len,d,k,vocab,dt", [(8, 128, 512, 40, 300, synth.BF16),
                                                      (32, 64, 256, 16, 100, synth.BF16),
                                                      (3, 50, 128, 5, 40, synth.BF16),
                                                      (2, 64, 128, 8, 30, synth.F32)])
def test_head_embed(batch, seq_len, d, k, vocab, dt):
    wl = synth.Workload("head", d, k, vocab, batch, seq_len, dt)
    t = synth.codec_inputs(wl, seed=batch + d)
    n = wl.n_tokens
    rng = np.random.default_rng(d + k)
    Elow0 = synth.to_storage(rng.standard_normal((vocab, k)), dt)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt), to_device(t["P"], dt))
    ids_np = t["ids"].copy()
    ids_np[1] = vocab                                   # one id outside both tables
    ids = torch.from_numpy(ids_np).cuda()
    X0 = codec.head_embed(to_device(Elow0, dt), ids, seq_len=seq_len)
    pos = oracle.token_positions(n, seq_len)
    expect, status = oracle.head_embed(f64(Elow0, dt), f64(t["U"], dt), f64(t["E"], dt), ids_np,
                                       f64(t["P"], dt), pos)
    assert_close(host64(X0, dt), expect, dt, "head embed")
    assert codec.take_status() == status == binding.SSN_DEV_BAD_ID
    # compressing the head input gives the rows of Elow back (lossless inside the subspace)
    good = np.ones(n, dtype=bool)
    good[1] = False
    Z = codec.compress(X0, ids, seq_len=seq_len)
    codec.take_status()
    assert_close(host64(Z, dt)[good], f64(Elow0, dt)[ids_np[good]], dt, "compress(head embed)", tol=2e-2 if dt == synth.BF16 else 1e-4)


@pytest.mark.parametrize("n,m,d,k,dt", CASES + [(65536, 4096, 4096, 40, synth.BF16), (1100, 200, 256, 24, synth.BF16)])
def test_reparam_grad_factor(n, m, d, k, dt):
    """dZw = H^T (dY U): tensor-core shapes (several CTAs per row block add their partial sums)
    and general ones, against the oracle."""
    if n * m > 1 << 28:
        pytest.skip("too large for the oracle in a unit test")
    rng = np.random.default_rng(n + m + 3 * d + k)
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=m + k), dt)
    H0 = synth.to_storage(rng.standard_normal((n, m)) * 0.5, dt)
    dY0 = synth.to_storage(rng.standard_normal((n, d)) * 0.01, dt)
    codec = Codec(dt, to_device(U0, dt))
    got = codec.reparam_grad_factor(to_device(H0, dt), to_device(dY0, dt))
    expect = oracle.reparam_grad_factor(f64(H0, dt), f64(dY0, dt), f64(U0, dt))
    assert_close(got.double().cpu().numpy(), expect, dt, "dZw = H^T (dY U)")
    # a second call overwrites, it does not accumulate
    got2 = codec.reparam_grad_factor(to_device(H0, dt), to_device(dY0, dt))
    assert_close(got2.double().cpu().numpy(), expect, dt, "second call")


def test_activation_gradient_is_the_same_call_with_the_factors_exchanged():
    """dH = (dY U) Zw^T: ssn_reparam_project on a codec whose basis is Zw, with U as the factor."""
    dt, n, m, d, k = synth.BF16, 1536, 1024, 512, 40
    rng = np.random.default_rng(7)
    U0 = synth.to_storage(synth.subspace_basis(d, k, seed=9), dt)
    Zw0 = synth.to_storage(rng.standard_normal((m, k)) / np.sqrt(m), dt)
    dY0 = synth.to_storage(rng.standard_normal((n, d)) * 0.01, dt)
    swapped = Codec(dt, to_device(Zw0, dt))              # "U" of this codec is Zw: [m x k]
    dH = swapped.reparam_project(to_device(dY0, dt), to_device(U0, dt))
    expect = (f64(dY0, dt) @ f64(U0, dt)) @ f64(Zw0, dt).T
    assert_close(host64(dH, dt), expect, dt, "dH = (dY U) Zw^T")


def test_reparam_argument_errors():
    dt, d, k = synth.BF16, 256, 8
    codec = Codec(dt, to_device(synth.to_storage(synth.subspace_basis(d, k, seed=3), dt), dt))
    H = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
    Zw = torch.zeros((64, k), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((16, d), dtype=torch.bfloat16, device="cuda")
    fn = binding.raw("ssn_reparam_project")
    ok = lambda *a: fn(codec.c, *a)
    assert ok(H.data_ptr(), 64, 64, Zw.data_ptr(), k, 16, Y.data_ptr(), d, None, 0, None) == binding.SSN_OK
    assert ok(H.data_ptr(), 63, 64, Zw.data_ptr(), k, 16, Y.data_ptr(), d, None, 0, None) == binding.SSN_ERR_SHAPE
    assert ok(H.data_ptr(), 64, 64, Zw.data_ptr(), k - 1, 16, Y.data_ptr(), d, None, 0, None) == binding.SSN_ERR_SHAPE
    assert ok(H.data_ptr(), 64, 64, Zw.data_ptr(), k, 16, Y.data_ptr(), d - 1, None, 0, None) == binding.SSN_ERR_SHAPE
    assert ok(None, 64, 64, Zw.data_ptr(), k, 16, Y.data_ptr(), d, None, 0, None) == binding.SSN_ERR_NULL
    assert ok(H.data_ptr(), 64, 64, Zw.data_ptr(), k, 0, Y.data_ptr(), d, None, 0, None) == binding.SSN_OK
    g = binding.raw("ssn_reparam_grad_factor")
    dZ = torch.zeros((64, k), dtype=torch.float32, device="cuda")
    ws = torch.zeros(16 * 8 * 2, dtype=torch.uint8, device="cuda")
    assert g(codec.c, H.data_ptr(), 64, 64, Y.data_ptr(), d, 16, dZ.data_ptr(), k, ws.data_ptr(), ws.numel(), None) == binding.SSN_OK
    assert g(codec.c, H.data_ptr(), 64, 64, Y.data_ptr(), d, 16, dZ.data_ptr(), k, None, 0, None) == binding.SSN_ERR_WORKSPACE
    assert g(codec.c, H.data_ptr(), 64, 64, Y.data_ptr(), d, 16, dZ.data_ptr(), k - 1, ws.data_ptr(), ws.numel(), None) == binding.SSN_ERR_SHAPE
    assert g(codec.c, H.data_ptr(), 64, 64, None, d, 16, dZ.data_ptr(), k, ws.data_ptr(), ws.numel(), None) == binding.SSN_ERR_NULL
    torch.cuda.synchronize()
