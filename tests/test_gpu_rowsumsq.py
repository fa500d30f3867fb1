"""GPU parity of ssn_decompress_rowsumsq (decompress fused with the RMSNorm row statistic of the
receiving stage's first block) against the oracle: the reconstruction within the codec's
tolerance, the statistic within 1e-5 relative (it is formed in fp32 from the unrounded values on
both paths), on the tcgen05 expansion kernel and on the general kernel."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding as B
from paper_2607_13332_b200 import synth
from tests.harness import Codec, assert_close, f64, guards_intact, host64, padded, to_device

pytestmark = pytest.mark.gpu

STAT_TOL = 1e-5


def _check(wl, tables, expect_family, pos_np=None, ld_pad=0, seed=3):
    t = synth.codec_inputs(wl, seed=seed, noise_std=1e-3)
    dt, n = wl.dtype, wl.n_tokens
    E0 = t["E"] if "E" in tables else None
    P0 = t["P"] if "P" in tables else None
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    pos = torch.from_numpy(pos_np).cuda() if pos_np is not None else None
    out, buf = padded(n, wl.d, wl.d + ld_pad, dt)
    stat = torch.full((n + 2,), 777.0, dtype=torch.float32, device="cuda")     # guard words at both ends
    codec.decompress_rowsumsq(to_device(t["Z0"], dt), ids, seq_len=wl.seq_len, pos=pos, out=out,
                              rowsumsq=stat[1:n + 1])
    fam, var = B.ssn_last_kernel()
    assert fam == expect_family and var & B.SSN_KVAR_ROWSUMSQ
    Xo, so, _ = oracle.decompress_rowsumsq(f64(t["Z0"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], f64(P0, dt),
                                           pos_np if pos_np is not None else oracle.token_positions(n, wl.seq_len))
    assert_close(host64(out, dt), Xo, dt, "reconstruction")
    got = stat[1:n + 1].double().cpu().numpy()
    assert_close(got, so, dt, "row sum of squares", tol=STAT_TOL)
    assert float(np.max(np.abs(got - so) / so)) <= 10 * STAT_TOL          # and row by row, plainly relative
    assert guards_intact(out, buf, dt)
    assert float(stat[0]) == 777.0 and float(stat[n + 1]) == 777.0
    assert codec.take_status() == 0


@pytest.mark.parametrize("k", [40, 72])
@pytest.mark.parametrize("tables", ["EP", "E", "P", "none"])
@pytest.mark.parametrize("batch,seq_len,d", [(8, 128, 256), (160, 128, 256), (16, 272, 1024)])
def test_rowsumsq_on_the_tcgen05_expansion(batch, seq_len, d, k, tables):
    """From 1024 tokens (below the large-batch limit, where the plain decompress would take the
    few-rows kernel) to 20480, one and two coordinate groups, every table combination."""
    wl = synth.Workload("stat", d, k, 700, batch, seq_len, synth.BF16, "zipf")
    _check(wl, tables, B.SSN_KERNEL_UMMA_EXPAND, ld_pad=64, seed=batch + k)


@pytest.mark.parametrize("batch,seq_len", [(2, 2048), (3, 1024), (6, 512)])
def test_rowsumsq_few_sequences_on_the_tcgen05_expansion(batch, seq_len):
    wl = synth.Workload("stat", 512, 40, 300, batch, seq_len, synth.BF16, "zipf")
    _check(wl, "EP", B.SSN_KERNEL_UMMA_EXPAND, ld_pad=8, seed=batch)


def test_rowsumsq_ragged_token_count_on_the_tcgen05_expansion():
    wl = synth.Workload("stat", 128, 24, 300, 1, 5 * 128 + 11, synth.BF16, "zipf")
    _check(wl, "E", B.SSN_KERNEL_UMMA_EXPAND, ld_pad=8)


@pytest.mark.parametrize("case", ["fp32", "explicit_pos", "odd_width", "few_tokens"])
def test_rowsumsq_on_the_general_kernel(case):
    if case == "fp32":
        wl = synth.TINY.scaled(batch=1)
        _check(wl, "EP", B.SSN_KERNEL_GENERIC)
    elif case == "explicit_pos":
        wl = synth.Workload("stat", 256, 40, 100, 8, 128, synth.BF16)
        pos_np = np.random.default_rng(4).integers(0, wl.seq_len, wl.n_tokens).astype(np.int32)
        _check(wl, "EP", B.SSN_KERNEL_GENERIC, pos_np=pos_np)
    elif case == "odd_width":
        wl = synth.Workload("stat", 200, 24, 100, 4, 160, synth.BF16)
        _check(wl, "EP", B.SSN_KERNEL_GENERIC)
    else:
        wl = synth.Workload("stat", 256, 16, 100, 1, 100, synth.BF16)
        _check(wl, "E", B.SSN_KERNEL_GENERIC)


def test_rowsumsq_argument_errors():
    wl = synth.Workload("stat", 128, 8, 20, 1, 64, synth.BF16)
    t = synth.codec_inputs(wl, seed=1)
    codec = Codec(wl.dtype, to_device(t["U"], wl.dtype))
    Z = to_device(t["Z0"], wl.dtype)
    X = torch.empty((64, 128), dtype=torch.bfloat16, device="cuda")
    fn = B.raw("ssn_decompress_rowsumsq")
    assert fn(codec.c, Z.data_ptr(), 8, None, None, 64, 1, X.data_ptr(), 128, None, None, None) == B.SSN_ERR_NULL
    assert fn(codec.c, Z.data_ptr(), 8, None, None, 0, 1, None, 128, None, None, None) == B.SSN_OK
    assert fn(codec.c, Z.data_ptr(), 7, None, None, 64, 1, X.data_ptr(), 128, 0x1000, None, None) == B.SSN_ERR_SHAPE
