"""Parity at the sizes the benchmark times: every point of the compress sweep (model width 1024 to
8192, rank 8 to 128, 4096 / 65536 / 524288 tokens, uniform ids over 128256) and the 8B-class
stage boundary at 524288 tokens, in the launch configuration the benchmark uses.  The oracle
computes the first and the last tile and 4096 seeded random tokens of every point, one by one;
every token is independent, so those rows are checked element by element."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding as B
from paper_2607_13332_b200 import synth, synth_device
from tests.harness import Codec, assert_close, to_host

pytestmark = pytest.mark.gpu

DT = synth.BF16
VOCAB, SEQ = synth_device.SWEEP_VOCAB, synth_device.SWEEP_SEQ_LEN


def _host64(t: torch.Tensor) -> np.ndarray:
    return synth.to_f64(to_host(t, DT), DT)


def _sampled_tables(E, P, ids_np, rows):
    """The E and P rows the sampled tokens need, as small float64 tables with local indices."""
    uniq, local = np.unique(ids_np[rows], return_inverse=True)
    Es = _host64(E[torch.from_numpy(uniq).to(E.device)])
    pos = rows % SEQ
    return Es, local.astype(np.int64), _host64(P), pos


@pytest.mark.parametrize("d", [1024, 2048, 4096, 8192])
def test_compress_sweep_points_against_sampled_oracle(d):
    gen = synth_device.generator(d)
    E = synth_device.embedding_table(VOCAB, d, gen)
    P = synth_device.positions_table(SEQ, d)
    for k in (8, 32, 64, 128):
        U = synth_device.basis(d, k, 1)
        Uf = _host64(U)
        codec, codec_t = Codec(DT, U, E, P), Codec(DT, U, E, P)
        codec_t.prepare_tables()
        for n in (4096, 65536, 524288):
            ids_np = synth_device.uniform_ids(n, VOCAB, n + d + k)
            ids = torch.from_numpy(ids_np).cuda()
            X = synth_device.activations(n, d, gen)
            rows = synth_device.sample_rows(n, seed=n + k)
            rows_dev = torch.from_numpy(rows).cuda()
            Es, local_ids, Pf, pos = _sampled_tables(E, P, ids_np, rows)
            Zo, _ = oracle.compress(_host64(X[rows_dev]), Uf, Es, local_ids, Pf, pos)
            for name, c in (("rows", codec), ("tables", codec_t)):
                Z = c.compress(X, ids, seq_len=SEQ)
                fam, _ = B.ssn_last_kernel()
                assert fam == B.SSN_KERNEL_UMMA_PROJECT
                assert_close(_host64(Z[rows_dev]), Zo, DT, f"compress {name} d={d} k={k} n={n}")
                assert c.take_status() == 0
            del X, ids


@pytest.mark.parametrize("n", [4096, 12288, 524288])
def test_stage_boundary_steps_at_benchmark_sizes(n):
    """d = 4096, k = 40, Zipf ids: decompress and grad-project beside compress, at the call sizes of
    the paper's per-stage timing table (1 to 3 coalesced sequences of 4096) and at 512K tokens."""
    d, k = 4096, 40
    gen = synth_device.generator(n)
    E = synth_device.embedding_table(VOCAB, d, gen)
    P = synth_device.positions_table(SEQ, d)
    U = synth_device.basis(d, k, 1)
    Uf = _host64(U)
    codec = Codec(DT, U, E, P)
    ids_np = synth.zipf_ids(n, VOCAB, 1.1, seed=n)
    ids = torch.from_numpy(ids_np).cuda()
    rows = synth_device.sample_rows(n, seed=n)
    rows_dev = torch.from_numpy(rows).cuda()
    Es, local_ids, Pf, pos = _sampled_tables(E, P, ids_np, rows)

    X = synth_device.activations(n, d, gen)
    Zo, _ = oracle.compress(_host64(X[rows_dev]), Uf, Es, local_ids, Pf, pos)
    assert_close(_host64(codec.compress(X, ids, seq_len=SEQ)[rows_dev]), Zo, DT, "compress")
    dZo = oracle.grad_project_coeff(_host64(X[rows_dev]), Uf)
    assert_close(_host64(codec.grad_project(X)[rows_dev]), dZo, DT, "grad-project")
    del X
    Z = synth_device.activations(n, k, gen)
    Xo, _ = oracle.decompress(_host64(Z[rows_dev]), Uf, Es, local_ids, Pf, pos)
    Xh = codec.decompress(Z, ids, seq_len=SEQ)
    assert_close(_host64(Xh[rows_dev]), Xo, DT, "decompress")
    assert codec.take_status() == 0
