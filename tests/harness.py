"""Shared plumbing of the GPU parity tests: upload stored tensors, call the C-ABI through the
binding, download, widen to float64 for comparison with the oracle."""

from __future__ import annotations

import numpy as np
import torch

from oracle import ssn_oracle as oracle
from oracle.metrics import max_rel_err
from paper_2607_13332_b200 import synth
from paper_2607_13332_b200.runner import Codec, to_device, to_host

TOL = {synth.F32: 1e-5, synth.BF16: 1e-2}   # max relative error (oracle.metrics.max_rel_err)
SENTINEL = {synth.F32: 12345.0, synth.BF16: 12288.0}


def f64(stored, dtype):
    return None if stored is None else synth.to_f64(stored, dtype)


def padded(rows: int, cols: int, ld: int, dtype: str, fill=None, guard_rows: int = 1):
    """A [rows, cols] view with leading dimension ld inside a sentinel-filled buffer that also
    has guard rows before and after; returns (view, whole buffer)."""
    tdt = torch.float32 if dtype == synth.F32 else torch.bfloat16
    buf = torch.full((rows + 2 * guard_rows, ld), SENTINEL[dtype], dtype=tdt, device="cuda")
    view = buf[guard_rows:guard_rows + rows, :cols]
    if fill is not None:
        view.copy_(fill)
    return view, buf


def guards_intact(view, buf, dtype, guard_rows: int = 1) -> bool:
    rows, cols = view.shape
    s = SENTINEL[dtype]
    ok = bool((buf[:guard_rows] == s).all()) and bool((buf[guard_rows + rows:] == s).all())
    if buf.shape[1] > cols:
        ok = ok and bool((buf[guard_rows:guard_rows + rows, cols:] == s).all())
    return ok


def host64(t: torch.Tensor, dtype: str) -> np.ndarray:
    return synth.to_f64(to_host(t, dtype), dtype)


def assert_close(got64, expect64, dtype, what, tol=None):
    err = max_rel_err(got64, expect64)
    limit = TOL[dtype] if tol is None else tol
    assert err <= limit, f"{what}: max rel err {err:.3e} > {limit:g}"
    return err
