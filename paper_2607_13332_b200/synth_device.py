"""Seeded inputs generated ON the device, for the sweep sizes at which the host generator of
``synth`` would need minutes and tens of GB of host memory (524288 tokens x 8192 columns).

Only value distributions live here (the same laws as ``synth``: activations ~ N(0, 1), the fixed
embedding ~ N(0, 0.02^2), uniform token ids); none of the codec's arithmetic.  The benchmark
sweeps and the full-size parity tests draw their inputs from this module, so both time and check
the same bytes; the tests download the sampled rows they hand to the oracle.
"""

from __future__ import annotations

import numpy as np
import torch

from . import synth

SWEEP_VOCAB = 128256
SWEEP_SEQ_LEN = 2048


def generator(seed: int, device: str = "cuda") -> torch.Generator:
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return gen


def embedding_table(vocab: int, d: int, gen: torch.Generator) -> torch.Tensor:
    """T_fixed stand-in [vocab x d], N(0, 0.02^2), bf16."""
    return (torch.randn((vocab, d), device=gen.device, generator=gen) * 0.02).bfloat16()


def activations(n: int, d: int, gen: torch.Generator, std: float = 1.0) -> torch.Tensor:
    """Dense rows [n x d], N(0, std^2), bf16, made in slabs so that the fp32 draw stays small."""
    out = torch.empty((n, d), dtype=torch.bfloat16, device=gen.device)
    step = max(1, (1 << 28) // d)
    for lo in range(0, n, step):
        hi = min(n, lo + step)
        out[lo:hi] = (torch.randn((hi - lo, d), device=gen.device, generator=gen) * std).bfloat16()
    return out


def uniform_ids(n: int, vocab: int, seed: int) -> np.ndarray:
    """Token ids uniform over the vocabulary (host array; the caller uploads it)."""
    return np.random.default_rng(seed).integers(0, vocab, n).astype(np.int32)


def positions_table(seq_len: int, d: int, device: str = "cuda") -> torch.Tensor:
    """The sinusoidal PE stand-in of ``synth`` [seq_len x d], uploaded as bf16."""
    bits = synth.to_storage(synth.sinusoidal_positions(seq_len, d), synth.BF16)
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def basis(d: int, k: int, seed: int, device: str = "cuda") -> torch.Tensor:
    """Orthonormal basis of ``synth`` [d x k], uploaded as bf16."""
    bits = synth.to_storage(synth.subspace_basis(d, k, seed), synth.BF16)
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def sample_rows(n: int, tile: int = 128, extra: int = 4096, seed: int = 0) -> np.ndarray:
    """Row indices for a sampled comparison: the first and last `tile` rows plus `extra` seeded
    random ones, sorted and unique."""
    if n <= 2 * tile + extra:
        return np.arange(n, dtype=np.int64)
    rnd = np.random.default_rng(seed).integers(tile, n - tile, extra)
    return np.unique(np.concatenate([np.arange(tile), rnd, np.arange(n - tile, n)])).astype(np.int64)
