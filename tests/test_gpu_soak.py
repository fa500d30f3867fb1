"""Back-to-back soak of the stage-boundary step at the benchmark's size.

The tcgen05 kernels hand stages between warps through mbarrier rings; a mistake in such a
handshake may show only once in many thousand launches, and only when loads complete out of their
usual order (for instance right after an idle gap, while clocks ramp).  Each case lets the device go
idle, queues several hundred steps without a host wait in between, and then checks that every
output still equals, bit for bit, what the first step wrote (the kernels are deterministic) and
that no wait ran out.  The element-by-element comparison with the oracle at this size is in
test_gpu_parity.py; this test is about the handshakes."""

import time

import pytest
import torch

from paper_2607_13332_b200 import synth, synth_device
from tests.harness import Codec

pytestmark = pytest.mark.gpu

DT = synth.BF16
D, SEQ, NSEQ = 4096, 2048, 32
STEPS, ROUNDS = 300, 4

# (rank, E rows, P rows, prepared tables): the benchmark's two step variants, then the projection
# kernel's other issuer layouts (E alone: four issuing threads on a ring of five; P alone; k = 128:
# accumulators of 128 columns, one set only when E and P are operands)
CASES = {
    "rows": (40, True, True, False),
    "prepared_tables": (40, True, True, True),
    "embedding_only": (40, True, False, False),
    "positions_only": (40, False, True, False),
    "rank_128": (128, True, True, False),
}


@pytest.mark.parametrize("case", list(CASES))
def test_queued_steps_after_idle_gaps_repeat_the_first_step(case):
    k, with_e, with_p, tables = CASES[case]
    n = SEQ * NSEQ
    gen = synth_device.generator(77)
    E = synth_device.embedding_table(synth_device.SWEEP_VOCAB, D, gen) if with_e else None
    P = synth_device.positions_table(SEQ, D) if with_p else None
    U = synth_device.basis(D, k, 1)
    X = synth_device.activations(n, D, gen)
    G = synth_device.activations(n, D, gen)
    ids = torch.from_numpy(synth.zipf_ids(n, synth_device.SWEEP_VOCAB, 1.1, seed=5)).cuda()
    codec = Codec(DT, U, E, P)
    if tables:
        codec.prepare_tables()
    Z = torch.empty((n, k), dtype=torch.bfloat16, device="cuda")
    dZ = torch.empty_like(Z)
    Xh = torch.empty_like(X)
    # the weights are re-projected in place step after step (projecting twice gives the same weight
    # only up to rounding, so they are checked for staying finite, not for equality)
    W = [synth_device.activations(r, D, gen) for r in (4096, 14336)]

    def step():
        codec.compress(X, ids, seq_len=SEQ, out=Z)
        codec.decompress(Z, ids, seq_len=SEQ, out=Xh)
        codec.grad_project(G, out=dZ)
        codec.weight_reproject_rows(W)

    step()
    torch.cuda.synchronize()
    first = [t.clone() for t in (Z, dZ, Xh)]
    for _ in range(ROUNDS):
        time.sleep(0.3)            # let the device drop to its idle clocks
        for _ in range(STEPS):
            step()
        torch.cuda.synchronize()
        assert codec.take_status() == 0
        for got, want in zip((Z, dZ, Xh), first):
            assert torch.equal(got, want)
        assert all(bool(torch.isfinite(w.float()).all()) for w in W)
