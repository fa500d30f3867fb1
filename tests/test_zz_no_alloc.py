"""The allocation-free LEFT re-projection (ssn_weight_reproject_left_static) against the regular
entry point.  Collected last on purpose: if it fails, everything else has already run.

Some callers cannot allocate device memory at call time (all of it belongs to an arena, or
cudaMalloc's implicit synchronisation is not acceptable); for them the library keeps the fp32
coordinates in a fixed internal array.  The results must be those of ssn_weight_reproject."""

import ctypes

import numpy as np
import pytest
import torch

from paper_2607_13332_b200 import synth
from tests.harness import Codec, host64, to_device
from oracle.metrics import max_rel_err

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dt", [synth.BF16, synth.F32])
def test_static_scratch_matches_regular_entry_point_twice(libssn, dt):
    b = libssn
    d, k = 512, 24
    U = to_device(synth.to_storage(synth.subspace_basis(d, k, seed=3), dt), dt)
    codec = Codec(dt, U)
    assert b.ssn_static_scratch_bytes() == 4 << 20
    # two calls in a row with different widths: the second must not see anything of the first.
    # Odd widths: with a leading dimension that is not a multiple of 8 the regular entry point
    # also takes its general two-kernel form, so the results can be compared bit for bit.
    for cols, seed in ((1001, 1), (333, 2)):
        W0 = synth.projection_weight(d, cols, seed=seed, dtype=dt)
        ref = to_device(W0, dt)
        codec.weight_reproject([ref], "left")
        got = to_device(W0, dt)
        b.ssn_weight_reproject_left_static(codec.c, got.data_ptr(), cols, cols,
                                           torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        tol = 1e-5 if dt == synth.F32 else 1e-2
        assert max_rel_err(host64(got, dt), host64(ref, dt)) <= tol
        assert torch.equal(got, ref)      # same kernels, same order of operations


def test_static_scratch_rejects_oversized_problems(libssn):
    b = libssn
    dt = synth.BF16
    d, k = 256, 128
    U = to_device(synth.to_storage(synth.subspace_basis(d, k, seed=4), dt), dt)
    codec = Codec(dt, U)
    cols = b.ssn_static_scratch_bytes() // (4 * k) + 1        # one column too many
    W = torch.zeros((d, cols), dtype=torch.bfloat16, device="cuda")
    fn = b.raw("ssn_weight_reproject_left_static")
    assert fn(ctypes.byref(codec.c), W.data_ptr(), cols, cols, None) == b.SSN_ERR_WORKSPACE
    with pytest.raises(b.SsnError) as err:
        b.ssn_weight_reproject_left_static(codec.c, W.data_ptr(), cols, cols)
    assert err.value.status == b.SSN_ERR_WORKSPACE and "workspace" in str(err.value)
    assert fn(ctypes.byref(codec.c), W.data_ptr(), cols - 1, cols, None) == b.SSN_OK
    torch.cuda.synchronize()
