"""Torch-tensor convenience layer over the ctypes binding.

Torch is used for device memory and streams only: every method below allocates the output,
hands raw addresses to the C-ABI call of the same name and returns.  No arithmetic happens in
Python and nothing here works without the CUDA library.
"""

from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding, synth

_TORCH_DTYPE = {synth.F32: torch.float32, synth.BF16: torch.bfloat16}


def to_device(stored: Optional[np.ndarray], dtype: str, device: str = "cuda") -> Optional[torch.Tensor]:
    """Upload a tensor kept in storage form (float32 array or uint16 bf16 bits)."""
    if stored is None:
        return None
    if dtype == synth.F32:
        return torch.from_numpy(np.ascontiguousarray(stored, dtype=np.float32)).to(device)
    bits = np.ascontiguousarray(stored, dtype=np.uint16).view(np.int16)
    return torch.from_numpy(bits).to(device).view(torch.bfloat16)


def to_host(t: torch.Tensor, dtype: str) -> np.ndarray:
    """Download to storage form (float32 array or uint16 bf16 bits)."""
    if dtype == synth.F32:
        return t.detach().cpu().numpy()
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def padded_columns(t: torch.Tensor, multiple: int = 8) -> torch.Tensor:
    """A copy of the 2-D tensor t whose leading dimension is rounded up to `multiple` elements,
    returned as the [rows, cols] view of the padded buffer (zeros in the padding).  The
    tensor-core kernels need such leading dimensions; see the note in include/ssn.h."""
    rows, cols = t.shape
    ld = -(-cols // multiple) * multiple
    buf = torch.zeros((rows, ld), dtype=t.dtype, device=t.device)
    buf[:, :cols] = t
    return buf[:, :cols]


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ld(t: torch.Tensor) -> int:
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("expected a row-major 2-D tensor (unit stride along the last dimension)")
    return max(t.stride(0), t.shape[1]) if t.shape[0] > 1 else t.shape[1]


class Codec:
    """The data both ends of a stage boundary share: U [d,k], optional E [V,d] and P [S,d]."""

    def __init__(self, dtype: str, U: torch.Tensor, E: Optional[torch.Tensor] = None,
                 P: Optional[torch.Tensor] = None):
        self.dtype = dtype
        self.U, self.E, self.P = U, E, P
        self.d, self.k = U.shape
        for t in (U, E, P):
            if t is not None and (not t.is_cuda or t.dtype != _TORCH_DTYPE[dtype]):
                raise ValueError("codec tensors must be CUDA tensors of the codec dtype")
        self.EU = self.PU = None
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=U.device)
        self.c = binding.make_codec(
            self.d, self.k, binding.DTYPES[dtype], U.data_ptr(), _ld(U),
            E.data_ptr() if E is not None else 0, _ld(E) if E is not None else None,
            E.shape[0] if E is not None else 0,
            P.data_ptr() if P is not None else 0, _ld(P) if P is not None else None,
            P.shape[0] if P is not None else 0, dev_status=self.dev_status.data_ptr())

    def prepare_tables(self, embedding: bool = True, positions: bool = True) -> None:
        """Project the codec's constant tables once (EU = E U, PU = P U, fp32) and attach them,
        so that compress reads k floats per token and table instead of the E and P rows.  Either
        table alone is allowed: PU is only seq_len x k and takes microseconds to make.  Call it
        again after changing U, E or P in place."""
        dev = self.U.device
        self.drop_tables()
        if embedding and self.E is not None:
            self.EU = torch.empty((self.E.shape[0], self.k), dtype=torch.float32, device=dev)
        if positions and self.P is not None:
            self.PU = torch.empty((self.P.shape[0], self.k), dtype=torch.float32, device=dev)
        binding.ssn_prepare_tables(self.c, self.EU.data_ptr() if self.EU is not None else 0, self.k,
                                   self.PU.data_ptr() if self.PU is not None else 0, self.k, _stream())
        if self.EU is not None:
            self.c.EU, self.c.ldeu = self.EU.data_ptr(), self.k
        if self.PU is not None:
            self.c.PU, self.c.ldpu = self.PU.data_ptr(), self.k

    def drop_tables(self) -> None:
        self.c.EU = self.c.PU = None
        self.EU = self.PU = None

    def _empty(self, rows: int, cols: int) -> torch.Tensor:
        return torch.empty((rows, cols), dtype=_TORCH_DTYPE[self.dtype], device=self.U.device)

    def take_status(self) -> int:
        """Read and clear the device status word (synchronises): SSN_DEV_BAD_ID, SSN_DEV_BAD_POS
        and SSN_DEV_TIMEOUT bits of every call made through this object since the last read."""
        v = int(self.dev_status.item())
        self.dev_status.zero_()
        return v

    @staticmethod
    def describe_status(status: int) -> str:
        names = [name for bit, name in ((binding.SSN_DEV_BAD_ID, "token id outside the table"),
                                        (binding.SSN_DEV_BAD_POS, "position outside the table"),
                                        (binding.SSN_DEV_TIMEOUT, "a kernel's bounded wait ran out: output invalid"))
                 if status & bit]
        return "; ".join(names) if names else "ok"

    def compress(self, X: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                 pos: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = X.shape[0]
        Z = out if out is not None else self._empty(n, self.k)
        binding.ssn_compress(self.c, X.data_ptr(), _ld(X), ids.data_ptr() if ids is not None else 0,
                             pos.data_ptr() if pos is not None else 0, n, seq_len, Z.data_ptr(),
                             _ld(Z), self.dev_status.data_ptr(), _stream())
        return Z

    def decompress(self, Z: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                   pos: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = Z.shape[0]
        Xh = out if out is not None else self._empty(n, self.d)
        binding.ssn_decompress(self.c, Z.data_ptr(), _ld(Z), ids.data_ptr() if ids is not None else 0,
                               pos.data_ptr() if pos is not None else 0, n, seq_len, Xh.data_ptr(),
                               _ld(Xh), self.dev_status.data_ptr(), _stream())
        return Xh

    def decompress_rowsumsq(self, Z: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                            pos: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                            rowsumsq: Optional[torch.Tensor] = None):
        """decompress plus the RMSNorm statistic of the rows it writes: (Xhat, sum_i Xhat[t,i]^2)."""
        n = Z.shape[0]
        Xh = out if out is not None else self._empty(n, self.d)
        ss = rowsumsq if rowsumsq is not None else torch.empty(n, dtype=torch.float32, device=self.U.device)
        binding.ssn_decompress_rowsumsq(self.c, Z.data_ptr(), _ld(Z), ids.data_ptr() if ids is not None else 0,
                                        pos.data_ptr() if pos is not None else 0, n, seq_len, Xh.data_ptr(),
                                        _ld(Xh), ss.data_ptr(), self.dev_status.data_ptr(), _stream())
        return Xh, ss

    def grad_project(self, G: torch.Tensor, full: bool = False, coeff: bool = True,
                     out: Optional[torch.Tensor] = None, out_full: Optional[torch.Tensor] = None):
        n = G.shape[0]
        mode = (binding.SSN_GRAD_COEFF if coeff else 0) | (binding.SSN_GRAD_FULL if full else 0)
        dZ = (out if out is not None else self._empty(n, self.k)) if coeff else None
        Gp = (out_full if out_full is not None else self._empty(n, self.d)) if full else None
        binding.ssn_grad_project(self.c, G.data_ptr(), _ld(G), n, mode,
                                 dZ.data_ptr() if coeff else 0, _ld(dZ) if coeff else 0,
                                 Gp.data_ptr() if full else 0, _ld(Gp) if full else 0, _stream())
        if coeff and full:
            return dZ, Gp
        return dZ if coeff else Gp

    # ---- wire rows: k fp32 coordinates (+ the token id as an int32 word) per token ------------
    def wire_buffer(self, n: int, with_ids: bool, ldw: Optional[int] = None) -> torch.Tensor:
        """An int32-typed [n, ldw] buffer of wire words (view the coordinates with .view(torch.float32))."""
        ldw = ldw if ldw is not None else self.k + (1 if with_ids else 0)
        return torch.empty((n, ldw), dtype=torch.int32, device=self.U.device)

    def compress_wire(self, X: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                      pos: Optional[torch.Tensor] = None, with_ids: bool = False,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = X.shape[0]
        wire = out if out is not None else self.wire_buffer(n, with_ids)
        binding.ssn_compress_wire(self.c, X.data_ptr(), _ld(X), ids.data_ptr() if ids is not None else 0,
                                  pos.data_ptr() if pos is not None else 0, n, seq_len, wire.data_ptr(),
                                  _ld(wire), with_ids, self.dev_status.data_ptr(), _stream())
        return wire

    def compress_sum(self, X: torch.Tensor, R: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                     pos: Optional[torch.Tensor] = None, wire: bool = False, with_ids: bool = False,
                     out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """compress(X + R) without forming the sum; Z in the storage dtype, or wire rows."""
        n = X.shape[0]
        if out is None:
            out = self.wire_buffer(n, with_ids) if wire else self._empty(n, self.k)
        form = (binding.SSN_OUT_WIRE_IDS if with_ids else binding.SSN_OUT_WIRE) if wire else binding.SSN_OUT_STORAGE
        binding.ssn_compress_sum(self.c, X.data_ptr(), _ld(X), R.data_ptr(), _ld(R),
                                 ids.data_ptr() if ids is not None else 0,
                                 pos.data_ptr() if pos is not None else 0, n, seq_len, out.data_ptr(), _ld(out),
                                 form, self.dev_status.data_ptr(), _stream())
        return out

    def grad_project_wire(self, G: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = G.shape[0]
        dZ = out if out is not None else torch.empty((n, self.k), dtype=torch.float32, device=self.U.device)
        binding.ssn_grad_project_wire(self.c, G.data_ptr(), _ld(G), n, dZ.data_ptr(), _ld(dZ), _stream())
        return dZ

    def decompress_wire(self, wire: torch.Tensor, ids: Optional[torch.Tensor] = None, seq_len: int = 1,
                        pos: Optional[torch.Tensor] = None, with_ids: bool = False,
                        out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                        use_workspace: bool = True) -> torch.Tensor:
        n = wire.shape[0]
        Xh = out if out is not None else self._empty(n, self.d)
        if workspace is None:
            nbytes = binding.ssn_decompress_wire_workspace_bytes(self.c, n, with_ids)
            if not use_workspace:   # only what the ids need: the general kernel runs
                nbytes = (n * 4 + 255) // 256 * 256 if with_ids else 0
            workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.U.device) if nbytes else None
        binding.ssn_decompress_wire(self.c, wire.data_ptr(), _ld(wire), with_ids,
                                    ids.data_ptr() if ids is not None else 0,
                                    pos.data_ptr() if pos is not None else 0, n, seq_len, Xh.data_ptr(), _ld(Xh),
                                    workspace.data_ptr() if workspace is not None else 0,
                                    workspace.numel() if workspace is not None else 0,
                                    self.dev_status.data_ptr(), _stream())
        return Xh

    def reproject_workspace(self, rows: int, cols: int, side: str, batch: int) -> Optional[torch.Tensor]:
        nbytes = binding.ssn_weight_reproject_workspace_bytes(self.c, rows, cols, binding.SIDES[side], batch)
        if nbytes == 0:
            return None
        return torch.empty(nbytes, dtype=torch.uint8, device=self.U.device)

    def reparam_project(self, H: torch.Tensor, Zw: torch.Tensor, out: Optional[torch.Tensor] = None,
                        coords: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Y = (H Zw) U^T for a projection stored as its factor Zw [m, k] (Eq. reparam)."""
        n, m = H.shape
        Y = out if out is not None else self._empty(n, self.d)
        binding.ssn_reparam_project(self.c, H.data_ptr(), _ld(H), m, Zw.data_ptr(), _ld(Zw), n, Y.data_ptr(),
                                    _ld(Y), coords.data_ptr() if coords is not None else 0,
                                    _ld(coords) if coords is not None else 0, _stream())
        return Y

    def reparam_grad_factor(self, H: torch.Tensor, dY: torch.Tensor) -> torch.Tensor:
        """dZw [m, k] (fp32) = H^T (dY U) for a projection stored as its factor (Eq. reparam)."""
        n, m = H.shape
        out = torch.empty((m, self.k), dtype=torch.float32, device=self.U.device)
        kpad = -(-self.k // 8) * 8
        ws = torch.empty(n * kpad * 4, dtype=torch.uint8, device=self.U.device)
        binding.ssn_reparam_grad_factor(self.c, H.data_ptr(), _ld(H), m, dY.data_ptr(), _ld(dY), n,
                                        out.data_ptr(), self.k, ws.data_ptr(), ws.numel(), _stream())
        return out

    def head_embed(self, Elow: torch.Tensor, ids: torch.Tensor, seq_len: int = 1,
                   pos: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """X0 = E[ids] + Elow[ids] U^T + P[pos]: the head stage's input with the factored embedding."""
        n = ids.shape[0]
        X0 = out if out is not None else self._empty(n, self.d)
        kpad = -(-self.k // 8) * 8
        ws = torch.empty(n * kpad * 4, dtype=torch.uint8, device=self.U.device)
        binding.ssn_head_embed(self.c, Elow.data_ptr(), _ld(Elow), Elow.shape[0], ids.data_ptr(),
                               pos.data_ptr() if pos is not None else 0, n, seq_len, X0.data_ptr(), _ld(X0),
                               ws.data_ptr(), ws.numel(), self.dev_status.data_ptr(), _stream())
        return X0

    def weight_reproject_list(self, weights: Sequence[torch.Tensor], side: str = "right",
                              workspace: Optional[torch.Tensor] = None) -> None:
        """In place, for weights [rows_i x d] ("right") or [d x cols_i] ("left") of any free
        extents.  A LEFT weight the fused kernel does not take needs k * cols * 4 bytes of workspace;
        one is allocated here when none is given."""
        if not weights:
            return
        axis = 0 if side == "right" else 1
        if side == "left" and workspace is None:
            workspace = torch.empty(self.k * max(w.shape[1] for w in weights) * 4, dtype=torch.uint8,
                                    device=self.U.device)
        binding.ssn_weight_reproject_list(self.c, [w.data_ptr() for w in weights],
                                          [w.shape[axis] for w in weights], [_ld(w) for w in weights],
                                          binding.SIDES[side],
                                          workspace.data_ptr() if workspace is not None else 0,
                                          workspace.numel() if workspace is not None else 0, _stream())

    def weight_reproject_rows(self, weights: Sequence[torch.Tensor]) -> None:
        self.weight_reproject_list(weights, "right")

    def weight_reproject(self, weights: Sequence[torch.Tensor], side: str,
                         workspace: Optional[torch.Tensor] = None) -> None:
        """In place, for a list of equally shaped weights."""
        if not weights:
            return
        rows, cols = weights[0].shape
        ldw = _ld(weights[0])
        for w in weights:
            if tuple(w.shape) != (rows, cols) or _ld(w) != ldw:
                raise ValueError("weights of one call must share shape and leading dimension")
        if workspace is None:
            workspace = self.reproject_workspace(rows, cols, side, len(weights))
        binding.ssn_weight_reproject(self.c, [w.data_ptr() for w in weights], rows, cols, ldw,
                                     binding.SIDES[side],
                                     workspace.data_ptr() if workspace is not None else 0,
                                     workspace.numel() if workspace is not None else 0, _stream())
