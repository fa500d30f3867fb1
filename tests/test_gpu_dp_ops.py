"""GPU parity of the data-parallel device ops (AsyncSPARTA round steps of Algorithm 3, Eq. sparta,
Eq. delta_rule; stage-wise clipping of Sec. 4.3) against the oracle."""

import numpy as np
import pytest
import torch

from oracle import dp_oracle as dp
from oracle.metrics import max_rel_err
from paper_2607_13332_b200 import binding, dp_ops

pytestmark = pytest.mark.gpu

F32_TOL = 1e-5


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def host(t):
    return t.cpu().numpy().astype(np.float64)


# parameter count, senders, round: vector path, ragged tails, unaligned segment starts, tiny
@pytest.mark.parametrize("n,senders,rnd", [(1 << 20, 4, 3), (1_000_003, 3, 7), (4099, 16, 19), (37, 2, 19),
                                             (20_000_000, 2, 11)])
def test_sparta_round(n, senders, rnd):
    rng = np.random.default_rng(n % 1000 + senders)
    lo, hi = dp_ops.sparta_segment(n, 20, rnd)
    assert (lo, hi) == dp.sparta_segment(n, 20, rnd)
    bufs0 = [rng.standard_normal(n).astype(np.float32) for _ in range(senders)]
    weights = [float(w) for w in rng.integers(0, 5, senders)]
    weights[0] = 2.0                                         # at least one contributes
    bufs = [dev(b) for b in bufs0]
    # every sender snapshots its segment; sender 0 is the reducer
    snaps = [dp_ops.sparta_snapshot(b, lo, hi) for b in bufs]
    for s, b0 in zip(snaps, bufs0):
        assert np.array_equal(s.cpu().numpy(), b0[lo:hi])    # a copy is bit-exact
    acc = torch.zeros(hi - lo, dtype=torch.float32, device="cuda")
    acc_o = np.zeros(hi - lo)
    for s, b0, w in zip(snaps, bufs0, weights):
        dp_ops.sparta_accumulate(acc, s, w)
        acc_o = dp.sparta_accumulate(acc_o, b0[lo:hi], w)
    assert max_rel_err(host(acc), acc_o) <= F32_TOL
    deltas = dp_ops.sparta_deltas(acc, sum(weights), snaps)
    mean_o, deltas_o = dp.sparta_deltas(acc_o, sum(weights), [b0[lo:hi] for b0 in bufs0])
    assert max_rel_err(host(acc), mean_o) <= F32_TOL
    for d_gpu, d_o in zip(deltas, deltas_o):
        assert max_rel_err(host(d_gpu), d_o) <= F32_TOL
    # the senders add their deltas: every buf[P] is the group average, the rest is untouched
    for b, b0, d_o in zip(bufs, bufs0, deltas_o):
        dp_ops.sparta_add_delta(b, lo, hi, dev(d_o))
        expect = dp.sparta_add_delta(b0, lo, hi, d_o.astype(np.float32))
        got = b.cpu().numpy()
        assert max_rel_err(got[lo:hi].astype(np.float64), expect[lo:hi]) <= F32_TOL
        assert np.array_equal(got[:lo], b0[:lo]) and np.array_equal(got[hi:], b0[hi:])
    # in-place deltas give the same values
    snaps2 = [dp_ops.sparta_snapshot(dev(b0), lo, hi) for b0 in bufs0]
    acc2 = dev(acc_o)
    out = dp_ops.sparta_deltas(acc2, sum(weights), snaps2, in_place=True)
    for d_gpu, d_o in zip(out, deltas_o):
        assert max_rel_err(host(d_gpu), d_o) <= F32_TOL


@pytest.mark.parametrize("n,lo,hi,lam", [(1 << 20, 1 << 18, 1 << 19, 1.0), (100_003, 5001, 77_778, 1.0),
                                          (50, 10, 30, 0.5), (64, 0, 64, 1.0), (64, 7, 7, 1.0)])
def test_sparta_apply_round(n, lo, hi, lam):
    rng = np.random.default_rng(n + lo)
    theta0 = rng.standard_normal(n).astype(np.float32)
    avg0 = rng.standard_normal(hi - lo).astype(np.float32)
    snap0 = rng.standard_normal(hi - lo).astype(np.float32)
    theta = dev(theta0)
    dp_ops.sparta_apply_round(theta, lo, hi, dev(avg0), dev(snap0), lam)
    expect = dp.sparta_apply_round(theta0, lo, hi, avg0, snap0, lam)
    got = theta.cpu().numpy()
    if hi > lo:
        assert max_rel_err(got[lo:hi].astype(np.float64), expect[lo:hi]) <= F32_TOL
    assert np.array_equal(got[:lo], theta0[:lo]) and np.array_equal(got[hi:], theta0[hi:])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("sizes,scale", [([1 << 20, 4099, 7], 1.0), ([1 << 20, 4099, 7], 1e-5), ([33], 3.0),
                                         ([5_000_001], 0.01)])
def test_stage_clip(dtype, sizes, scale):
    """Several tensors of one stage, one of them starting off a 16-byte boundary; a gradient
    outside the budget is scaled to the threshold, one inside it is left bit-identical."""
    rng = np.random.default_rng(sum(sizes) % 977)
    thr = binding.stage_clip_threshold(7, False)
    assert abs(thr - dp.stage_clip_threshold(7, False)) < 1e-7
    assert abs(binding.stage_clip_threshold(7, True) - dp.stage_clip_threshold(7, True)) < 1e-7
    pool = torch.empty(sum(sizes) + 8 * len(sizes) + 1, dtype=dtype, device="cuda")
    grads, off = [], 1                                       # offset 1: the first tensor is unaligned
    for sz in sizes:
        g = pool[off:off + sz]
        g.copy_(torch.from_numpy((rng.standard_normal(sz) * scale).astype(np.float32)).cuda())
        grads.append(g)
        off += sz + (-sz % 8) + 8
    before = [g.clone() for g in grads]
    stored = [b.float().cpu().numpy().astype(np.float64) for b in before]
    expect, norm, coef = dp.stage_clip(stored, thr)
    sumsq = dp_ops.stage_clip(grads, thr)
    assert abs(float(sumsq.item()) - norm * norm) <= 1e-6 * norm * norm   # squares summed four (eight) at a time in fp32
    tol = F32_TOL if dtype == torch.float32 else 1e-2
    for g, b, e in zip(grads, before, expect):
        if coef == 1.0:
            assert torch.equal(g, b)
        else:
            assert max_rel_err(g.float().cpu().numpy().astype(np.float64), e) <= tol
    if coef < 1.0 and dtype == torch.float32:
        new_norm = np.sqrt(sum(float((g.double() ** 2).sum().item()) for g in grads))
        assert abs(new_norm - thr) < 1e-5


def test_dp_ops_argument_errors():
    a = torch.zeros(16, dtype=torch.float32, device="cuda")
    for call, status in (
            (lambda: binding.sparta_segment(100, 0, 1), binding.SSN_ERR_SHAPE),
            (lambda: binding.sparta_snapshot(a.data_ptr(), 5, 4, a.data_ptr()), binding.SSN_ERR_SHAPE),
            (lambda: binding.sparta_snapshot(0, 0, 4, a.data_ptr()), binding.SSN_ERR_NULL),
            (lambda: binding.sparta_accumulate(a.data_ptr(), 0, 1.0, 4), binding.SSN_ERR_NULL),
            (lambda: binding.sparta_deltas(a.data_ptr(), 0.0, [a.data_ptr()], [a.data_ptr()], 4), binding.SSN_ERR_SHAPE),
            (lambda: binding.sparta_deltas(a.data_ptr(), 1.0, [a.data_ptr()] * 17, [a.data_ptr()] * 17, 4),
             binding.SSN_ERR_SHAPE),
            (lambda: binding.sparta_deltas(a.data_ptr(), 1.0, [0], [a.data_ptr()], 4), binding.SSN_ERR_NULL),
            (lambda: binding.stage_clip_sumsq(a.data_ptr(), 4, 9, a.data_ptr()), binding.SSN_ERR_DTYPE),
            (lambda: binding.stage_clip_scale(a.data_ptr(), 4, 0, a.data_ptr(), 0.0), binding.SSN_ERR_SHAPE),
            (lambda: binding.stage_clip_sumsq(a.data_ptr(), 4, 0, 0), binding.SSN_ERR_NULL)):
        with pytest.raises(binding.SsnError) as e:
            call()
        assert e.value.status == status
    binding.sparta_accumulate(0, 0, 1.0, 0)                   # empty calls are no-ops
    binding.sparta_snapshot(0, 3, 3, 0)
    assert binding.stage_clip_threshold(0, False) == 0.0
