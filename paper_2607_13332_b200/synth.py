"""Seeded synthetic inputs for the SSN stage-boundary codec.

This module serves both the CUDA path (tests, benchmark) and the CPU oracle's tests.  It
holds storage-format plumbing (bf16 bit patterns kept as ``uint16``) and the statement of the
synthetic workloads -- shapes, value laws, id distributions -- and nothing else: it calls
neither the oracle nor the CUDA library.

The workloads stand in for the paper's activations (Sec. 4.1): a residual stream that is an
embedding row plus a positional row plus a point of the shared k-dimensional subspace,
``X = E[ids] + P[pos] + Z0 U^T``, optionally with a little off-subspace noise.  Only the
shapes (d, k, vocabulary, sequence length) and the skew of natural token frequencies are
borrowed from the paper's 8B-class run; all values are random.

Random numbers come from numpy's Philox counter-based generator, so a (seed, stream) pair
names the same tensor on every machine.
"""

from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

F32 = "f32"
BF16 = "bf16"


# --------------------------------------------------------------------------------------
# storage formats
# --------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (round-to-nearest-even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    rounded = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float array to the storage dtype: float32 array, or uint16 bf16 bit patterns."""
    if dtype == F32:
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == BF16:
        return f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    raise ValueError(f"unknown storage dtype {dtype!r}")


def to_f64(stored: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of a stored tensor to float64 (what the oracle consumes)."""
    if dtype == F32:
        return np.asarray(stored, dtype=np.float32).astype(np.float64)
    if dtype == BF16:
        return bf16_bits_to_f32(stored).astype(np.float64)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def itemsize(dtype: str) -> int:
    return {F32: 4, BF16: 2}[dtype]


# --------------------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    """One stage-boundary workload: X is [batch*seq_len, d] token-major, U is [d, k]."""

    name: str
    d: int
    k: int
    vocab: int
    batch: int
    seq_len: int
    dtype: str
    ids_law: str = "uniform"  # "uniform" or "zipf"
    zipf_s: float = 1.1

    @property
    def n_tokens(self) -> int:
        return self.batch * self.seq_len

    def scaled(self, batch: int) -> "Workload":
        """Same workload with fewer (or more) sequences; everything else unchanged."""
        return replace(self, batch=batch)


#: The three codec workloads the benchmark definition lists (tiny / mid / 8B-class boundary).
TINY = Workload("tiny", d=512, k=8, vocab=1024, batch=4, seq_len=1024, dtype=F32)
MID = Workload("mid", d=2048, k=32, vocab=32000, batch=16, seq_len=2048, dtype=BF16)
STAGE_8B = Workload("stage8b", d=4096, k=40, vocab=128256, batch=32, seq_len=2048, dtype=BF16,
                    ids_law="zipf", zipf_s=1.1)
WORKLOADS = {w.name: w for w in (TINY, MID, STAGE_8B)}

#: Weight shapes of the re-projection sweep at d=4096 (rows, cols): attention out-projection
#: and MLP down-projection, the latter with d last (rows of W lie in the subspace).
REPROJECT_SHAPES_8B = {"out_proj": (4096, 4096), "down_proj": (14336, 4096)}
REPROJECT_RANKS = (16, 40, 64, 128)

_STREAMS = {"U": 1, "E": 2, "ids": 3, "perm": 4, "Z0": 5, "noise": 6, "G": 7, "W": 8, "X": 9}


def _rng(seed: int, stream: str, index: int = 0) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | (_STREAMS[stream] << 32) | (int(index) << 40)
    return np.random.Generator(np.random.Philox(key=key))


def subspace_basis(d: int, k: int, seed: int) -> np.ndarray:
    """Orthonormal basis [d, k] in float64: thin QR of a seeded Gaussian, diag(R) > 0."""
    a = _rng(seed, "U").standard_normal((d, k))
    q, r = np.linalg.qr(a)
    sign = np.sign(np.diag(r))
    sign[sign == 0] = 1.0
    return q * sign[None, :]


def sinusoidal_positions(max_pos: int, d: int) -> np.ndarray:
    """Standard sinusoidal table [max_pos, d] in float64 (the paper gives no formula for PE)."""
    pos = np.arange(max_pos, dtype=np.float64)[:, None]
    i = np.arange(0, d, 2, dtype=np.float64)[None, :]
    angle = pos / np.power(10000.0, i / d)
    table = np.zeros((max_pos, d), dtype=np.float64)
    table[:, 0::2] = np.sin(angle)
    table[:, 1::2] = np.cos(angle)[:, : table[:, 1::2].shape[1]]
    return table


def embedding_table(vocab: int, d: int, seed: int, dtype: str, std: float = 0.02) -> np.ndarray:
    """Fixed token-embedding table [vocab, d] ~ N(0, std^2), already in the storage dtype."""
    rows_per_chunk = max(1, (1 << 24) // d)
    out = np.empty((vocab, d), dtype=np.float32 if dtype == F32 else np.uint16)
    rng = _rng(seed, "E")
    for lo in range(0, vocab, rows_per_chunk):
        hi = min(vocab, lo + rows_per_chunk)
        chunk = rng.standard_normal((hi - lo, d), dtype=np.float32) * np.float32(std)
        out[lo:hi] = to_storage(chunk, dtype)
    return out


def uniform_ids(n: int, vocab: int, seed: int) -> np.ndarray:
    return _rng(seed, "ids").integers(0, vocab, size=n, dtype=np.int64).astype(np.int32)


def zipf_ids(n: int, vocab: int, s: float, seed: int, scatter: bool = True) -> np.ndarray:
    """Token ids with Pr[rank r] proportional to r^-s, r = 1..vocab (inverse CDF in float64).

    With ``scatter`` the rank -> id map is a seeded permutation, so that the frequent rows
    are spread over the table as in a real vocabulary; otherwise rank r is id r-1.
    """
    weights = np.power(np.arange(1, vocab + 1, dtype=np.float64), -float(s))
    cdf = np.cumsum(weights)
    cdf /= cdf[-1]
    u = _rng(seed, "ids").random(n)
    ranks = np.minimum(np.searchsorted(cdf, u, side="right"), vocab - 1)
    if scatter:
        perm = _rng(seed, "perm").permutation(vocab)
        return perm[ranks].astype(np.int32)
    return ranks.astype(np.int32)


def token_ids(wl: Workload, seed: int) -> np.ndarray:
    if wl.ids_law == "uniform":
        return uniform_ids(wl.n_tokens, wl.vocab, seed)
    if wl.ids_law == "zipf":
        return zipf_ids(wl.n_tokens, wl.vocab, wl.zipf_s, seed)
    raise ValueError(wl.ids_law)


def default_positions(n_tokens: int, seq_len: int) -> np.ndarray:
    """Position of token t in a batch-major [batch, seq_len] flattening: t mod seq_len."""
    return (np.arange(n_tokens, dtype=np.int64) % seq_len).astype(np.int32)


def codec_inputs(wl: Workload, seed: int = 0x5EED, noise_std: float = 0.0,
                 with_positions: bool = True, grad_std: float = 1e-2,
                 make_grad: bool = True) -> Dict[str, Optional[np.ndarray]]:
    """All tensors of one codec workload, in the storage dtype of ``wl``.

    Returns U [d,k], E [vocab,d], P [seq_len,d] (or None), ids [n] int32, Z0 [n,k],
    X [n,d] = E[ids] + P[t mod seq_len] + Z0 U^T (+ N(0, noise_std^2)), and G [n,d] ~
    N(0, grad_std^2), the upstream activation-gradient.  X is assembled from the *stored*
    (already rounded) U, E, P and Z0 and rounded once more, so it lies in the shifted
    subspace up to its own storage rounding.
    """
    n, d, k, dt = wl.n_tokens, wl.d, wl.k, wl.dtype
    U = to_storage(subspace_basis(d, k, seed), dt)
    E = embedding_table(wl.vocab, d, seed, dt)
    P = to_storage(sinusoidal_positions(wl.seq_len, d), dt) if with_positions else None
    ids = token_ids(wl, seed)
    Z0 = to_storage(_rng(seed, "Z0").standard_normal((n, k), dtype=np.float32), dt)

    Uf = to_f64(U, dt)
    Ef32 = E if dt == F32 else bf16_bits_to_f32(E)
    Pf = to_f64(P, dt) if P is not None else None
    X = np.empty((n, d), dtype=np.float32 if dt == F32 else np.uint16)
    G = np.empty_like(X) if make_grad else None
    tokens_per_chunk = max(1, (1 << 23) // d)
    for c, lo in enumerate(range(0, n, tokens_per_chunk)):
        hi = min(n, lo + tokens_per_chunk)
        x = to_f64(Z0[lo:hi], dt) @ Uf.T
        x += Ef32[ids[lo:hi]]
        if Pf is not None:
            x += Pf[np.arange(lo, hi) % wl.seq_len]
        if noise_std > 0.0:
            x += _rng(seed, "noise", c).standard_normal((hi - lo, d), dtype=np.float32) * noise_std
        X[lo:hi] = to_storage(x, dt)
        if make_grad:
            g = _rng(seed, "G", c).standard_normal((hi - lo, d), dtype=np.float32)
            G[lo:hi] = to_storage(g * np.float32(grad_std), dt)
    return {"U": U, "E": E, "P": P, "ids": ids, "Z0": Z0, "X": X, "G": G}


def dense_activations(n: int, d: int, seed: int, dtype: str, std: float = 1.0) -> np.ndarray:
    """A generic [n, d] N(0, std^2) tensor with no subspace structure (stress input)."""
    out = np.empty((n, d), dtype=np.float32 if dtype == F32 else np.uint16)
    rows_per_chunk = max(1, (1 << 23) // d)
    for c, lo in enumerate(range(0, n, rows_per_chunk)):
        hi = min(n, lo + rows_per_chunk)
        x = _rng(seed, "X", c).standard_normal((hi - lo, d), dtype=np.float32) * np.float32(std)
        out[lo:hi] = to_storage(x, dtype)
    return out


def projection_weight(rows: int, cols: int, seed: int, dtype: str, layer: int = 0,
                      std: float = 0.02) -> np.ndarray:
    """One output-projection weight [rows, cols] ~ N(0, std^2) in the storage dtype."""
    out = np.empty((rows, cols), dtype=np.float32 if dtype == F32 else np.uint16)
    rng = _rng(seed, "W", layer)
    rows_per_chunk = max(1, (1 << 23) // cols)
    for lo in range(0, rows, rows_per_chunk):
        hi = min(rows, lo + rows_per_chunk)
        w = rng.standard_normal((hi - lo, cols), dtype=np.float32) * np.float32(std)
        out[lo:hi] = to_storage(w, dtype)
    return out


def shard_tokens(n_tokens: int, rank: int, world_size: int) -> range:
    """Contiguous token range of ``rank`` when n_tokens are split over ``world_size`` ranks.

    Tokens are independent in every codec step, so ranks never exchange data; the first
    ``n_tokens % world_size`` ranks take one extra token.
    """
    if not (0 <= rank < world_size):
        raise ValueError("rank out of range")
    base, extra = divmod(n_tokens, world_size)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))
