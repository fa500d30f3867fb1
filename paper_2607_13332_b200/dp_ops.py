"""Torch-tensor sugar over the data-parallel device ops of the C ABI (include/agora_dp.h):
argument marshalling only, every step runs in the library's kernels."""

from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding
from .runner import _stream


def _flat_f32(t: torch.Tensor) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise ValueError("expected a contiguous fp32 CUDA tensor")
    return t


def sparta_segment(n_params: int, rounds_per_cycle: int, rnd: int):
    return binding.sparta_segment(n_params, rounds_per_cycle, rnd)


def sparta_snapshot(buf: torch.Tensor, lo: int, hi: int) -> torch.Tensor:
    snap = torch.empty(hi - lo, dtype=torch.float32, device=buf.device)
    binding.sparta_snapshot(_flat_f32(buf).data_ptr(), lo, hi, snap.data_ptr(), _stream())
    return snap


def sparta_accumulate(acc: torch.Tensor, chunk: torch.Tensor, w: float) -> None:
    binding.sparta_accumulate(_flat_f32(acc).data_ptr(), _flat_f32(chunk).data_ptr(), w, acc.numel(), _stream())


def sparta_deltas(acc: torch.Tensor, sum_w: float, chunks: Sequence[torch.Tensor], in_place: bool = False) -> List[torch.Tensor]:
    """acc /= sum_w; returns [acc - c_i] (written over the chunks when in_place)."""
    deltas = list(chunks) if in_place else [torch.empty_like(c) for c in chunks]
    binding.sparta_deltas(_flat_f32(acc).data_ptr(), sum_w, [_flat_f32(c).data_ptr() for c in chunks],
                          [d.data_ptr() for d in deltas], acc.numel(), _stream())
    return deltas


def sparta_add_delta(buf: torch.Tensor, lo: int, hi: int, delta: torch.Tensor) -> None:
    binding.sparta_add_delta(_flat_f32(buf).data_ptr(), lo, hi, _flat_f32(delta).data_ptr(), _stream())


def sparta_apply_round(theta: torch.Tensor, lo: int, hi: int, avg: torch.Tensor, snap: torch.Tensor,
                       lam: float = 1.0) -> None:
    binding.sparta_apply_round(_flat_f32(theta).data_ptr(), lo, hi, _flat_f32(avg).data_ptr(),
                               _flat_f32(snap).data_ptr(), lam, _stream())


def stage_clip(grads: Sequence[torch.Tensor], threshold: float, sumsq: torch.Tensor = None) -> torch.Tensor:
    """Clips the stage's gradient tensors (fp32 or bf16, contiguous) in place by their joint norm;
    returns the device double holding the squared norm before clipping."""
    if sumsq is None:
        sumsq = torch.zeros(1, dtype=torch.float64, device=grads[0].device)
    else:
        sumsq.zero_()
    codes = {torch.float32: binding.DTYPES["f32"], torch.bfloat16: binding.DTYPES["bf16"]}
    for g in grads:
        if not (g.is_cuda and g.is_contiguous() and g.dtype in codes):
            raise ValueError("expected contiguous fp32 / bf16 CUDA gradients")
        binding.stage_clip_sumsq(g.data_ptr(), g.numel(), codes[g.dtype], sumsq.data_ptr(), _stream())
    for g in grads:
        binding.stage_clip_scale(g.data_ptr(), g.numel(), codes[g.dtype], sumsq.data_ptr(), threshold, _stream())
    return sumsq
