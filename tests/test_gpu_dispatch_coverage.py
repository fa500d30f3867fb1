"""GPU parity above the token count where the dispatch stops using the few-rows-per-SM kernels:
every kernel family (and template variant) that the large-batch calls of the benchmark reach is
run here at more than 18944 tokens, at a small model width so that the whole oracle stays
cheap, compared with the oracle element by element, and the test asserts WHICH kernel ran
(ssn_last_kernel), so the dispatch cannot drift away from what is checked."""

import numpy as np
import pytest
import torch

from oracle import ssn_oracle as oracle
from paper_2607_13332_b200 import binding as B
from paper_2607_13332_b200 import synth
from tests.harness import Codec, assert_close, f64, guards_intact, host64, padded, to_device, to_host

pytestmark = pytest.mark.gpu

LARGE = 148 * 8 * 16     # the dispatch's "few rows" limit on a 148-SM part: all cases are above it


def last_kernel():
    return B.ssn_last_kernel()


def expect_kernel(family, has=0, lacks=0):
    fam, var = last_kernel()
    assert fam == family, f"kernel family {fam}, expected {family} (variant bits {var:#x})"
    assert var & has == has and var & lacks == 0, f"variant bits {var:#x}: want {has:#x} set, {lacks:#x} clear"


def _inputs(batch, seq_len, d, k, vocab, seed, tables):
    wl = synth.Workload("cover", d, k, vocab, batch, seq_len, synth.BF16, "zipf")
    assert wl.n_tokens > LARGE
    t = synth.codec_inputs(wl, seed=seed, noise_std=1e-3)
    E0 = t["E"] if "E" in tables else None
    P0 = t["P"] if "P" in tables else None
    return wl, t, E0, P0


def _variant_bits(tables):
    return (B.SSN_KVAR_E if "E" in tables else 0) | (B.SSN_KVAR_P if "P" in tables else 0)


# ---- decompress on the tcgen05 expansion kernel: every template variant --------------------------
@pytest.mark.parametrize("k", [40, 72, 128])
@pytest.mark.parametrize("tables", ["EP", "E", "P", "none"])
@pytest.mark.parametrize("batch,seq_len", [(160, 128), (80, 272)])
def test_decompress_tcgen05_whole_sequences(batch, seq_len, k, tables):
    """Groups of 8 whole sequences whose length is a multiple of 16: with P the tiles are 8
    sequences x 16 positions, without P 128 consecutive tokens; one and two coordinate groups."""
    d = 256
    wl, t, E0, P0 = _inputs(batch, seq_len, d, k, 900, seed=batch + k, tables=tables)
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    out, buf = padded(n, d, d + 64, dt)
    codec.decompress(to_device(t["Z0"], dt), ids, seq_len=seq_len, out=out)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND,
                  has=_variant_bits(tables) | (B.SSN_KVAR_WIDE if k > 64 else 0) | (B.SSN_KVAR_ALT if P0 is not None else 0),
                  lacks=(B.SSN_KVAR_E | B.SSN_KVAR_P) & ~_variant_bits(tables) | (0 if k > 64 else B.SSN_KVAR_WIDE))
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], f64(P0, dt),
                              oracle.token_positions(n, seq_len))
    assert_close(host64(out, dt), Xo, dt, f"decompress {tables} k={k}")
    assert guards_intact(out, buf, dt)
    assert codec.take_status() == 0


@pytest.mark.parametrize("k", [40, 128])
@pytest.mark.parametrize("tables", ["E", "none"])
def test_decompress_tcgen05_ragged_last_tile(k, tables):
    """No positional table: tiles of 128 consecutive tokens, the last one with 11 live rows that
    the TMA store has to clip."""
    d, n = 128, 160 * 128 + 11
    wl, t, E0, P0 = _inputs(1, n, d, k, 300, seed=k, tables=tables)
    dt = wl.dtype
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    out, buf = padded(n, d, d + 8, dt, guard_rows=130)
    codec.decompress(to_device(t["Z0"], dt), ids, out=out)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND, has=_variant_bits(tables) | (B.SSN_KVAR_WIDE if k > 64 else 0),
                  lacks=B.SSN_KVAR_ALT | B.SSN_KVAR_P)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], None, None)
    assert_close(host64(out, dt), Xo, dt, f"decompress ragged {tables} k={k}")
    assert guards_intact(out, buf, dt, guard_rows=130)
    assert codec.take_status() == 0


@pytest.mark.parametrize("batch,seq_len", [(161, 128), (1, 2560), (2, 1280), (3, 1024), (4, 640), (6, 512), (12, 1728),
                                           (166, 128)])
@pytest.mark.parametrize("tables,k", [("EP", 40), ("P", 64), ("EP", 8)])
def test_decompress_tcgen05_few_sequences(batch, seq_len, tables, k):
    """Batches that are not groups of 8 sequences (the 1 to 6 sequences of a small call): tiles of
    4, 2 or 1 sequences x 32, 64 or 128 positions, whose P rows enter through a wider selection
    matrix.  From 2560 tokens (below the large-batch limit) to 21248."""
    # below the large-batch limit the dispatch takes the tcgen05 expansion for wide models only
    d = 256 if batch > 100 else (1024 if batch * seq_len > LARGE else 2048)
    wl = synth.Workload("few", d, k, 500, batch, seq_len, synth.BF16, "zipf")
    t = synth.codec_inputs(wl, seed=batch + k, noise_std=1e-3)
    dt, n = wl.dtype, wl.n_tokens
    E0 = t["E"] if "E" in tables else None
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(t["P"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    out, buf = padded(n, d, d + 64, dt)
    codec.decompress(to_device(t["Z0"], dt), ids, seq_len=seq_len, out=out)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND, has=_variant_bits(tables) | B.SSN_KVAR_ALT | B.SSN_KVAR_FEWSEQ)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], f64(t["P"], dt),
                              oracle.token_positions(n, seq_len))
    assert_close(host64(out, dt), Xo, dt, f"decompress {batch} x {seq_len} {tables} k={k}")
    assert guards_intact(out, buf, dt)
    assert codec.take_status() == 0


# ---- decompress on the mma.sync kernels the tcgen05 expansion hands over to ----------------------
@pytest.mark.parametrize("case", ["batch_not_8", "ragged_length", "explicit_pos", "d192_dedup", "d192_noshift",
                                  "d160", "d160_wide", "k72_explicit_pos"])
def test_decompress_mma_sync_large_batches(case):
    batch, seq_len, d, k, tables, explicit = {
        "batch_not_8": (161, 128, 256, 72, "EP", False),        # odd batch and a rank above 64
        "ragged_length": (1, 160 * 128 + 11, 256, 24, "EP", False),   # length not a multiple of 16
        "explicit_pos": (160, 128, 256, 40, "EP", True),        # positions given per token
        "d192_dedup": (160, 128, 192, 40, "EP", False),         # d % 128 != 0, 16-sequence tiles share a P row
        "d192_noshift": (160, 128, 192, 16, "none", False),
        "d160": (160, 128, 160, 40, "EP", False),               # d % 64 != 0: the 32-column kernel, 32 rows per warp
        "d160_wide": (160, 128, 160, 96, "E", False),           # and its wide-rank variant
        "k72_explicit_pos": (160, 128, 256, 72, "P", True),     # rank above 64 with explicit positions
    }[case]
    wl, t, E0, P0 = _inputs(batch, seq_len, d, k, 500, seed=len(case), tables=tables)
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    pos_np = oracle.token_positions(n, seq_len)
    if explicit:
        pos_np = np.random.default_rng(1).integers(0, seq_len, n).astype(np.int32)
    pos = torch.from_numpy(pos_np).cuda() if explicit else None
    out, buf = padded(n, d, d + 32, dt)
    codec.decompress(to_device(t["Z0"], dt), ids, seq_len=seq_len, pos=pos, out=out)
    want = {
        "batch_not_8": (B.SSN_KERNEL_MMA_SYNC, B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_WIDE, 0),
        "ragged_length": (B.SSN_KERNEL_EXPAND64, B.SSN_KVAR_E | B.SSN_KVAR_P, B.SSN_KVAR_ALT),
        "explicit_pos": (B.SSN_KERNEL_EXPAND64, B.SSN_KVAR_E | B.SSN_KVAR_P, B.SSN_KVAR_ALT),
        "d192_dedup": (B.SSN_KERNEL_EXPAND64, B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_ALT, 0),
        "d192_noshift": (B.SSN_KERNEL_EXPAND64, 0, B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_ALT),
        "d160": (B.SSN_KERNEL_MMA_SYNC, B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_ALT, B.SSN_KVAR_WIDE),
        "d160_wide": (B.SSN_KERNEL_MMA_SYNC, B.SSN_KVAR_E | B.SSN_KVAR_WIDE, B.SSN_KVAR_ALT | B.SSN_KVAR_P),
        "k72_explicit_pos": (B.SSN_KERNEL_MMA_SYNC, B.SSN_KVAR_P | B.SSN_KVAR_WIDE, B.SSN_KVAR_E),
    }[case]
    expect_kernel(*want)
    Xo, _ = oracle.decompress(f64(t["Z0"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], f64(P0, dt), pos_np)
    assert_close(host64(out, dt), Xo, dt, f"decompress {case}")
    assert guards_intact(out, buf, dt)
    assert codec.take_status() == 0


# ---- the projections and the fused form on the large-batch mma.sync kernel -----------------------
@pytest.mark.parametrize("k", [24, 104])
def test_project_and_roundtrip_mma_sync_large_batches(k):
    """d = 160 is no multiple of 64, so neither tcgen05 projection nor the fused kernel take it."""
    wl, t, E0, P0 = _inputs(160, 128, 160, k, 400, seed=k, tables="EP")
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    U, pos = f64(t["U"], dt), oracle.token_positions(n, wl.seq_len)
    Z = codec.compress(to_device(t["X"], dt), ids, seq_len=wl.seq_len)
    expect_kernel(B.SSN_KERNEL_MMA_SYNC, has=B.SSN_KVAR_E | B.SSN_KVAR_P | (B.SSN_KVAR_WIDE if k > 64 else B.SSN_KVAR_ALT))
    Zo, _ = oracle.compress(f64(t["X"], dt), U, f64(E0, dt), t["ids"], f64(P0, dt), pos)
    assert_close(host64(Z, dt), Zo, dt, "compress")
    dZ, Gp = codec.grad_project(to_device(t["G"], dt), full=True)
    expect_kernel(B.SSN_KERNEL_MMA_SYNC, lacks=B.SSN_KVAR_E | B.SSN_KVAR_P)
    assert_close(host64(dZ, dt), oracle.grad_project_coeff(f64(t["G"], dt), U), dt, "grad coeff")
    assert_close(host64(Gp, dt), oracle.grad_project_full(f64(t["G"], dt), U), dt, "grad full")
    assert codec.take_status() == 0


# ---- the projection kernel at large batches: shared positional product, ragged tail ---------------
# (widths of 1 and 3 stages: a tile whose second issuing threads get no stage of their own, and an
# odd number of stages for the two threads of an operand and for the two CTAs of a pair to share)
@pytest.mark.parametrize("d", [64, 192, 256])
@pytest.mark.parametrize("tables", ["EP", "E", "P", "none"])
def test_compress_tcgen05_large_batches(tables, d):
    wl, t, E0, P0 = _inputs(160, 128, d, 40, 900, seed=3, tables=tables)
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    Zv, Zbuf = padded(n, wl.k, wl.k + 8, dt)
    codec.compress(to_device(t["X"], dt), ids, seq_len=wl.seq_len, out=Zv)
    expect_kernel(B.SSN_KERNEL_UMMA_PROJECT,
                  has=_variant_bits(tables) | (B.SSN_KVAR_ALT if tables == "EP" else 0))
    Zo, _ = oracle.compress(f64(t["X"], dt), f64(t["U"], dt), f64(E0, dt), t["ids"], f64(P0, dt),
                            oracle.token_positions(n, wl.seq_len))
    assert_close(host64(Zv, dt), Zo, dt, f"compress {tables}")
    assert guards_intact(Zv, Zbuf, dt)
    assert codec.take_status() == 0


# ---- wire rows and the head-stage input above the limit -------------------------------------------
@pytest.mark.parametrize("k,with_ids", [(40, True), (40, False), (24, True), (24, False)])
def test_decompress_wire_large_batches(k, with_ids):
    """The fp32 coordinates travel as a bf16 head and a bf16 remainder, two products against the
    same chunk of U on the tcgen05 expansion."""
    wl, t, E0, P0 = _inputs(160, 128, 256, k, 700, seed=k + with_ids, tables="EP")
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    rng = np.random.default_rng(k)
    wire_np = oracle.wire_rows(rng.standard_normal((n, k)), t["ids"] if with_ids else None)
    coords, _ = oracle.wire_unpack(wire_np, k, with_ids)     # the fp32 words as the receiver sees them
    wire = torch.from_numpy(wire_np).cuda()
    ids = torch.from_numpy(t["ids"]).cuda()
    Xh = codec.decompress_wire(wire, None if with_ids else ids, seq_len=wl.seq_len, with_ids=with_ids)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND, has=B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_ALT | B.SSN_KVAR_TWO_RUNS,
                  lacks=B.SSN_KVAR_WIDE)
    Xo, _ = oracle.decompress(coords, f64(t["U"], dt), f64(E0, dt), t["ids"], f64(P0, dt),
                              oracle.token_positions(n, wl.seq_len))
    assert_close(host64(Xh, dt), Xo, dt, f"decompress_wire k={k}")
    assert codec.take_status() == 0


def test_head_embed_large_batch_with_a_bad_id():
    wl, t, E0, P0 = _inputs(160, 128, 256, 40, 600, seed=11, tables="EP")
    dt, n = wl.dtype, wl.n_tokens
    codec = Codec(dt, to_device(t["U"], dt), to_device(E0, dt), to_device(P0, dt))
    Elow0 = synth.to_storage(np.random.default_rng(2).standard_normal((wl.vocab, wl.k)), dt)
    ids_np = t["ids"].copy()
    ids_np[[5, n - 1]] = [wl.vocab, -3]
    X0 = codec.head_embed(to_device(Elow0, dt), torch.from_numpy(ids_np).cuda(), seq_len=wl.seq_len)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND, has=B.SSN_KVAR_E | B.SSN_KVAR_P | B.SSN_KVAR_ALT)
    Xo, flags = oracle.head_embed(f64(Elow0, dt), f64(t["U"], dt), f64(E0, dt), ids_np, f64(P0, dt),
                                  oracle.token_positions(n, wl.seq_len))
    assert_close(host64(X0, dt), Xo, dt, "head_embed")
    assert codec.take_status() == flags == B.SSN_DEV_BAD_ID


# ---- the gathered rows are bit-exact on the tcgen05 kernels too -----------------------------------
@pytest.mark.parametrize("d,k", [(256, 40), (128, 72)])
def test_gathered_rows_are_bit_exact_on_the_tcgen05_kernels(d, k):
    """Z = 0, no positional table: the expansion kernel hands back E[ids] bit for bit (a stored -0
    may come back as +0); X = E[ids] compresses to exactly zero on the projection kernel."""
    dt = synth.BF16
    wl = synth.Workload("gather", d, k, 700, 1, LARGE + 333, dt, "zipf")
    t = synth.codec_inputs(wl, seed=5, with_positions=False)
    codec = Codec(dt, to_device(t["U"], dt), to_device(t["E"], dt))
    ids = torch.from_numpy(t["ids"]).cuda()
    zero = torch.zeros((wl.n_tokens, k), dtype=torch.bfloat16, device="cuda")
    Xh = to_host(codec.decompress(zero, ids), dt)
    expect_kernel(B.SSN_KERNEL_UMMA_EXPAND, has=B.SSN_KVAR_E, lacks=B.SSN_KVAR_P)
    rows = t["E"][t["ids"]]
    both_zero = (f64(Xh, dt) == 0) & (f64(rows, dt) == 0)
    assert bool(np.all((Xh == rows) | both_zero))
    Z = codec.compress(to_device(rows, dt), ids)
    expect_kernel(B.SSN_KERNEL_UMMA_PROJECT, has=B.SSN_KVAR_E)
    assert bool((Z == 0).all())
    assert codec.take_status() == 0


# ---- the bounded waits --------------------------------------------------------------------------
def test_a_wait_that_runs_out_sets_the_timeout_bit_and_the_context_survives():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.ssn_selftest_bounded_wait(1000, status.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(status.item()) == B.SSN_DEV_TIMEOUT
    # the device still works, and a normal call leaves the bit clear
    wl = synth.Workload("after", 256, 16, 50, 8, 128, synth.BF16)
    t = synth.codec_inputs(wl, seed=1)
    codec = Codec(wl.dtype, to_device(t["U"], wl.dtype))
    dZ = codec.grad_project(to_device(t["G"], wl.dtype))
    assert_close(host64(dZ, wl.dtype), oracle.grad_project_coeff(f64(t["G"], wl.dtype), f64(t["U"], wl.dtype)),
                 wl.dtype, "grad after the self-test")
    assert codec.take_status() == 0


def test_two_devices_in_one_process():
    """The per-kernel shared-memory attribute is per device: a second GPU must work after the first."""
    if torch.cuda.device_count() < 2:
        pytest.skip("one GPU visible")
    wl = synth.Workload("dev", 256, 40, 50, 8, 128, synth.BF16)
    t = synth.codec_inputs(wl, seed=1)
    Zo = oracle.grad_project_coeff(f64(t["G"], wl.dtype), f64(t["U"], wl.dtype))
    for dev in (0, 1):
        with torch.cuda.device(dev):
            codec = Codec(wl.dtype, to_device(t["U"], wl.dtype, f"cuda:{dev}"))
            dZ = codec.grad_project(to_device(t["G"], wl.dtype, f"cuda:{dev}"))
            assert_close(host64(dZ, wl.dtype), Zo, wl.dtype, f"device {dev}")
