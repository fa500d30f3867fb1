"""ctypes binding of libssn: the same names as the C-ABI, argument marshalling only.

Every function takes raw device addresses (``tensor.data_ptr()``), sizes and a stream handle
(``torch.cuda.current_stream().cuda_stream``) and forwards them; all arithmetic happens in the
library's kernels.  Importing this module loads ``libssn.so`` from the package directory and
raises ``ImportError`` if it has not been built -- there is no CPU fallback.
"""

from __future__ import annotations

import ctypes
import os
import re
from typing import Optional, Sequence

from . import buildlib

SSN_OK = 0
SSN_ERR_NULL, SSN_ERR_SHAPE, SSN_ERR_DTYPE, SSN_ERR_WORKSPACE, SSN_ERR_CUDA = 1, 2, 3, 4, 5
SSN_F32, SSN_BF16 = 0, 1
SSN_SIDE_LEFT, SSN_SIDE_RIGHT = 0, 1
SSN_GRAD_COEFF, SSN_GRAD_FULL = 1, 2
SSN_DEV_BAD_ID, SSN_DEV_BAD_POS, SSN_DEV_TIMEOUT = 1, 2, 4
# ssn_last_kernel(): family | variant bits << 8
(SSN_KERNEL_NONE, SSN_KERNEL_GENERIC, SSN_KERNEL_MMA_SYNC, SSN_KERNEL_MMA_SYNC_DSPLIT, SSN_KERNEL_EXPAND64,
 SSN_KERNEL_UMMA_PROJECT, SSN_KERNEL_UMMA_EXPAND, SSN_KERNEL_UMMA_ROUNDTRIP, SSN_KERNEL_UMMA_TOKENS) = range(9)
SSN_KVAR_E, SSN_KVAR_P, SSN_KVAR_WIDE, SSN_KVAR_ALT, SSN_KVAR_ROWSUMSQ, SSN_KVAR_FEWSEQ, SSN_KVAR_TWO_RUNS = 1, 2, 4, 8, 16, 32, 64

DTYPES = {"f32": SSN_F32, "bf16": SSN_BF16}
SIDES = {"left": SSN_SIDE_LEFT, "right": SSN_SIDE_RIGHT}


class SsnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class ssn_codec_t(ctypes.Structure):
    _fields_ = [
        ("d", ctypes.c_int32), ("k", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("max_pos", ctypes.c_int32),
        ("U", ctypes.c_void_p), ("ldu", ctypes.c_int64),
        ("E", ctypes.c_void_p), ("lde", ctypes.c_int64), ("vocab", ctypes.c_int64),
        ("P", ctypes.c_void_p), ("ldp", ctypes.c_int64),
        ("EU", ctypes.c_void_p), ("ldeu", ctypes.c_int64),
        ("PU", ctypes.c_void_p), ("ldpu", ctypes.c_int64),
        ("dev_status", ctypes.c_void_p),
    ]


def _load() -> ctypes.CDLL:
    path = buildlib.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
            "(the SSN codec runs only through its CUDA library)")
    return ctypes.CDLL(path)


_lib = _load()
LIB_PATH = buildlib.LIB_PATH

_vp, _i64, _i32, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
_codec_p = ctypes.POINTER(ssn_codec_t)
_SIGNATURES = {
    "ssn_compress": (_i32, [_codec_p, _vp, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _vp, _vp]),
    "ssn_decompress": (_i32, [_codec_p, _vp, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _vp, _vp]),
    "ssn_decompress_rowsumsq": (_i32, [_codec_p, _vp, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _vp, _vp, _vp]),
    "ssn_grad_project": (_i32, [_codec_p, _vp, _i64, _i64, _i32, _vp, _i64, _vp, _i64, _vp]),
    "ssn_weight_reproject_workspace_bytes": (_sz, [_codec_p, _i64, _i64, _i32, _i32]),
    "ssn_weight_reproject": (_i32, [_codec_p, ctypes.POINTER(_vp), _i32, _i64, _i64, _i64, _i32,
                                    _vp, _sz, _vp]),
    "ssn_weight_reproject_left_static": (_i32, [_codec_p, _vp, _i64, _i64, _vp]),
    "ssn_prepare_tables": (_i32, [_codec_p, _vp, _i64, _vp, _i64, _vp]),
    "ssn_reparam_project": (_i32, [_codec_p, _vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _i64, _vp]),
    "ssn_reparam_grad_factor": (_i32, [_codec_p, _vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _sz, _vp]),
    "ssn_head_embed": (_i32, [_codec_p, _vp, _i64, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _vp, _sz, _vp, _vp]),
    "ssn_compress_wire": (_i32, [_codec_p, _vp, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _i32, _vp, _vp]),
    "ssn_compress_sum": (_i32, [_codec_p, _vp, _i64, _vp, _i64, _vp, _vp, _i64, _i32, _vp, _i64, _i32, _vp, _vp]),
    "ssn_grad_project_wire": (_i32, [_codec_p, _vp, _i64, _i64, _vp, _i64, _vp]),
    "ssn_decompress_wire_workspace_bytes": (_sz, [_codec_p, _i64, _i32]),
    "ssn_decompress_wire": (_i32, [_codec_p, _vp, _i64, _i32, _vp, _vp, _i64, _i32, _vp, _i64, _vp, _sz,
                                   _vp, _vp]),
    "ssn_weight_reproject_list": (_i32, [_codec_p, ctypes.POINTER(_vp), ctypes.POINTER(_i64),
                                         ctypes.POINTER(_i64), _i32, _i32, _vp, _sz, _vp]),
    "ssn_static_scratch_bytes": (_sz, []),
    "sparta_segment": (_i32, [_i64, _i32, _i64, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "sparta_snapshot": (_i32, [_vp, _i64, _i64, _vp, _vp]),
    "sparta_accumulate": (_i32, [_vp, _vp, ctypes.c_float, _i64, _vp]),
    "sparta_deltas": (_i32, [_vp, ctypes.c_float, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _i32, _i64, _vp]),
    "sparta_add_delta": (_i32, [_vp, _i64, _i64, _vp, _vp]),
    "sparta_apply_round": (_i32, [_vp, _i64, _i64, _vp, _vp, ctypes.c_float, _vp]),
    "stage_clip_threshold": (ctypes.c_float, [_i32, _i32]),
    "stage_clip_sumsq": (_i32, [_vp, _i64, _i32, _vp, _vp]),
    "stage_clip_scale": (_i32, [_vp, _i64, _i32, _vp, ctypes.c_float, _vp]),
    "ssn_status_string": (ctypes.c_char_p, [_i32]),
    "ssn_version": (_i32, []),
    "ssn_launch_count": (_i64, []),
    "ssn_last_kernel": (_i32, []),
    "ssn_selftest_bounded_wait": (_i32, [_i32, _vp, _vp]),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.restype, _fn.argtypes = _res, _args


def declared_symbols(header_dir: Optional[str] = None):
    """Names of the functions the public headers declare (parsed from include/*.h)."""
    header_dir = header_dir or os.path.join(buildlib.ROOT, "include")
    names = []
    for fname in sorted(os.listdir(header_dir)):
        if fname.endswith(".h"):
            text = open(os.path.join(header_dir, fname)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b((?:ssn|sparta|stage_clip)_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def status_string(status: int) -> str:
    return _lib.ssn_status_string(int(status)).decode()


def version() -> int:
    return int(_lib.ssn_version())


def ssn_launch_count() -> int:
    return int(_lib.ssn_launch_count())


def ssn_last_kernel():
    """(family, variant bits) of the calling thread's most recent codec launch."""
    code = int(_lib.ssn_last_kernel())
    return code & 0xFF, code >> 8


def ssn_selftest_bounded_wait(max_polls: int, dev_status: int, stream: int = 0) -> None:
    """One tiny kernel whose bounded wait runs out: ORs SSN_DEV_TIMEOUT into *dev_status."""
    _check(_lib.ssn_selftest_bounded_wait(max_polls, dev_status or None, stream or None),
           "ssn_selftest_bounded_wait")


def make_codec(d: int, k: int, dtype: int, U: int, ldu: Optional[int] = None, E: int = 0,
               lde: Optional[int] = None, vocab: int = 0, P: int = 0,
               ldp: Optional[int] = None, max_pos: int = 0, dev_status: int = 0) -> ssn_codec_t:
    """Fill an ``ssn_codec_t`` from raw device addresses (0 = NULL = term absent)."""
    return ssn_codec_t(d=d, k=k, dtype=dtype, max_pos=max_pos, U=U or None,
                       ldu=k if ldu is None else ldu, E=E or None,
                       lde=d if lde is None else lde, vocab=vocab, P=P or None,
                       ldp=d if ldp is None else ldp, dev_status=dev_status or None)


def _check(status: int, where: str) -> None:
    if status != SSN_OK:
        raise SsnError(status, where)


def ssn_compress(codec: ssn_codec_t, X: int, ldx: int, ids: int, pos: int, n_tokens: int,
                 seq_len: int, Z: int, ldz: int, dev_status: int = 0, stream: int = 0) -> None:
    _check(_lib.ssn_compress(ctypes.byref(codec), X or None, ldx, ids or None, pos or None,
                             n_tokens, seq_len, Z or None, ldz, dev_status or None,
                             stream or None), "ssn_compress")


def ssn_decompress(codec: ssn_codec_t, Z: int, ldz: int, ids: int, pos: int, n_tokens: int,
                   seq_len: int, Xhat: int, ldx: int, dev_status: int = 0, stream: int = 0) -> None:
    _check(_lib.ssn_decompress(ctypes.byref(codec), Z or None, ldz, ids or None, pos or None,
                               n_tokens, seq_len, Xhat or None, ldx, dev_status or None,
                               stream or None), "ssn_decompress")


def ssn_decompress_rowsumsq(codec: ssn_codec_t, Z: int, ldz: int, ids: int, pos: int, n_tokens: int,
                            seq_len: int, Xhat: int, ldx: int, rowsumsq: int, dev_status: int = 0,
                            stream: int = 0) -> None:
    """ssn_decompress that also writes rowsumsq[t] = sum_i Xhat[t,i]^2 (fp32, before rounding)."""
    _check(_lib.ssn_decompress_rowsumsq(ctypes.byref(codec), Z or None, ldz, ids or None, pos or None,
                                        n_tokens, seq_len, Xhat or None, ldx, rowsumsq or None,
                                        dev_status or None, stream or None), "ssn_decompress_rowsumsq")


def ssn_grad_project(codec: ssn_codec_t, G: int, ldg: int, n_tokens: int, mode: int, dZ: int = 0,
                     ldz: int = 0, Gpar: int = 0, ldgp: int = 0, stream: int = 0) -> None:
    _check(_lib.ssn_grad_project(ctypes.byref(codec), G or None, ldg, n_tokens, mode, dZ or None,
                                 ldz, Gpar or None, ldgp, stream or None), "ssn_grad_project")


def ssn_weight_reproject_workspace_bytes(codec: ssn_codec_t, rows: int, cols: int, side: int,
                                         batch: int) -> int:
    return int(_lib.ssn_weight_reproject_workspace_bytes(ctypes.byref(codec), rows, cols, side, batch))


def ssn_weight_reproject(codec: ssn_codec_t, W_ptrs: Sequence[int], rows: int, cols: int, ldw: int,
                         side: int, workspace: int = 0, workspace_bytes: int = 0,
                         stream: int = 0) -> None:
    arr = (_vp * max(1, len(W_ptrs)))(*[p or None for p in W_ptrs])
    _check(_lib.ssn_weight_reproject(ctypes.byref(codec), arr, len(W_ptrs), rows, cols, ldw, side,
                                     workspace or None, workspace_bytes, stream or None),
           "ssn_weight_reproject")


def ssn_static_scratch_bytes() -> int:
    return int(_lib.ssn_static_scratch_bytes())


def ssn_weight_reproject_left_static(codec: ssn_codec_t, W: int, cols: int, ldw: int,
                                     stream: int = 0) -> None:
    """LEFT re-projection of one weight [d x cols] using the library's fixed scratch array: for
    callers that cannot allocate or lend a workspace.  Raises SsnError(SSN_ERR_WORKSPACE) when
    k * cols * 4 exceeds ssn_static_scratch_bytes()."""
    _check(_lib.ssn_weight_reproject_left_static(ctypes.byref(codec), W or None, cols, ldw,
                                                 stream or None), "ssn_weight_reproject_left_static")


def ssn_weight_reproject_list(codec: ssn_codec_t, W_ptrs, extent, ldw, side: int, workspace: int = 0,
                              workspace_bytes: int = 0, stream: int = 0) -> None:
    """Re-projection of weights [extent[i] x d] (RIGHT) or [d x extent[i]] (LEFT), in place."""
    n = len(W_ptrs)
    _check(_lib.ssn_weight_reproject_list(ctypes.byref(codec), (_vp * n)(*W_ptrs), (_i64 * n)(*extent),
                                          (_i64 * n)(*ldw), n, side, workspace or None, workspace_bytes,
                                          stream or None), "ssn_weight_reproject_list")


def ssn_reparam_project(codec: ssn_codec_t, H: int, ldh: int, m: int, Zw: int, ldzw: int, n_tokens: int,
                        Y: int, ldy: int, coords: int = 0, ldc: int = 0, stream: int = 0) -> None:
    """Y [n x d] = (H [n x m] Zw [m x k]) U^T (Eq. reparam), optionally also the coordinates H Zw."""
    _check(_lib.ssn_reparam_project(ctypes.byref(codec), H or None, ldh, m, Zw or None, ldzw, n_tokens,
                                    Y or None, ldy, coords or None, ldc, stream or None),
           "ssn_reparam_project")


def ssn_reparam_grad_factor(codec: ssn_codec_t, H: int, ldh: int, m: int, dY: int, lddy: int, n_tokens: int,
                            dZw: int, lddz: int, workspace: int, workspace_bytes: int, stream: int = 0) -> None:
    """dZw [m x k] (fp32) = H^T (dY U): the gradient of a reparameterized projection's factor."""
    _check(_lib.ssn_reparam_grad_factor(ctypes.byref(codec), H or None, ldh, m, dY or None, lddy, n_tokens,
                                        dZw or None, lddz, workspace or None, workspace_bytes, stream or None),
           "ssn_reparam_grad_factor")


def ssn_head_embed(codec: ssn_codec_t, Elow: int, ldel: int, vocab_low: int, ids: int, pos: int,
                   n_tokens: int, seq_len: int, X0: int, ldx: int, workspace: int, workspace_bytes: int,
                   dev_status: int = 0, stream: int = 0) -> None:
    """X0[t] = E[ids[t]] + Elow[ids[t]] U^T + P[pos(t)] (head-stage input of the reparameterized SSN)."""
    _check(_lib.ssn_head_embed(ctypes.byref(codec), Elow or None, ldel, vocab_low, ids or None, pos or None,
                               n_tokens, seq_len, X0 or None, ldx, workspace or None, workspace_bytes,
                               dev_status or None, stream or None), "ssn_head_embed")


def ssn_compress_wire(codec: ssn_codec_t, X: int, ldx: int, ids: int, pos: int, n_tokens: int, seq_len: int,
                      wire: int, ldw: int, with_ids: bool, dev_status: int = 0, stream: int = 0) -> None:
    """ssn_compress into wire rows: k fp32 coordinates, then (with_ids) the token id as int32."""
    _check(_lib.ssn_compress_wire(ctypes.byref(codec), X or None, ldx, ids or None, pos or None, n_tokens,
                                  seq_len, wire or None, ldw, 1 if with_ids else 0, dev_status or None,
                                  stream or None), "ssn_compress_wire")


SSN_OUT_STORAGE, SSN_OUT_WIRE, SSN_OUT_WIRE_IDS = 0, 1, 2


def ssn_compress_sum(codec: ssn_codec_t, X: int, ldx: int, R: int, ldr: int, ids: int, pos: int, n_tokens: int,
                     seq_len: int, out: int, ldout: int, out_form: int = SSN_OUT_STORAGE, dev_status: int = 0,
                     stream: int = 0) -> None:
    """Z = (X + R - P[pos] - E[ids]) U: compress fused with the stage's last residual add."""
    _check(_lib.ssn_compress_sum(ctypes.byref(codec), X or None, ldx, R or None, ldr, ids or None, pos or None,
                                 n_tokens, seq_len, out or None, ldout, out_form, dev_status or None,
                                 stream or None), "ssn_compress_sum")


def ssn_grad_project_wire(codec: ssn_codec_t, G: int, ldg: int, n_tokens: int, dZ: int, ldw: int,
                          stream: int = 0) -> None:
    """dZ = G U as fp32 wire rows."""
    _check(_lib.ssn_grad_project_wire(ctypes.byref(codec), G or None, ldg, n_tokens, dZ or None, ldw,
                                      stream or None), "ssn_grad_project_wire")


def ssn_decompress_wire_workspace_bytes(codec: ssn_codec_t, n_tokens: int, with_ids: bool) -> int:
    return int(_lib.ssn_decompress_wire_workspace_bytes(ctypes.byref(codec), n_tokens, 1 if with_ids else 0))


def ssn_decompress_wire(codec: ssn_codec_t, wire: int, ldw: int, with_ids: bool, ids: int, pos: int,
                        n_tokens: int, seq_len: int, Xhat: int, ldx: int, workspace: int, workspace_bytes: int,
                        dev_status: int = 0, stream: int = 0) -> None:
    """ssn_decompress from wire rows (the ids come from the rows when with_ids)."""
    _check(_lib.ssn_decompress_wire(ctypes.byref(codec), wire or None, ldw, 1 if with_ids else 0, ids or None,
                                    pos or None, n_tokens, seq_len, Xhat or None, ldx, workspace or None,
                                    workspace_bytes, dev_status or None, stream or None), "ssn_decompress_wire")


def ssn_prepare_tables(codec: ssn_codec_t, EU: int, ldeu: int, PU: int, ldpu: int,
                       stream: int = 0) -> None:
    """EU [vocab x k] = E U and PU [max_pos x k] = P U in fp32 (0 = do not make that table)."""
    _check(_lib.ssn_prepare_tables(ctypes.byref(codec), EU or None, ldeu, PU or None, ldpu,
                                   stream or None), "ssn_prepare_tables")


def raw(name: str):
    """The raw ctypes function (returns the status instead of raising); used by error tests."""
    return getattr(_lib, name)


# ---- data-parallel device ops (include/agora_dp.h) --------------------------------------------
def sparta_segment(n_params: int, rounds_per_cycle: int, rnd: int):
    lo, hi = _i64(0), _i64(0)
    _check(_lib.sparta_segment(n_params, rounds_per_cycle, rnd, ctypes.byref(lo), ctypes.byref(hi)), "sparta_segment")
    return int(lo.value), int(hi.value)


def sparta_snapshot(buf: int, lo: int, hi: int, snap: int, stream: int = 0) -> None:
    _check(_lib.sparta_snapshot(buf or None, lo, hi, snap or None, stream or None), "sparta_snapshot")


def sparta_accumulate(acc: int, chunk: int, w: float, count: int, stream: int = 0) -> None:
    _check(_lib.sparta_accumulate(acc or None, chunk or None, w, count, stream or None), "sparta_accumulate")


def sparta_deltas(acc: int, sum_w: float, chunks, deltas, count: int, stream: int = 0) -> None:
    n = len(chunks)
    c_arr = (_vp * max(n, 1))(*chunks)
    d_arr = (_vp * max(n, 1))(*deltas)
    _check(_lib.sparta_deltas(acc or None, sum_w, c_arr, d_arr, n, count, stream or None), "sparta_deltas")


def sparta_add_delta(buf: int, lo: int, hi: int, delta: int, stream: int = 0) -> None:
    _check(_lib.sparta_add_delta(buf or None, lo, hi, delta or None, stream or None), "sparta_add_delta")


def sparta_apply_round(theta: int, lo: int, hi: int, avg: int, snap: int, lam: float = 1.0, stream: int = 0) -> None:
    _check(_lib.sparta_apply_round(theta or None, lo, hi, avg or None, snap or None, lam, stream or None),
           "sparta_apply_round")


def stage_clip_threshold(n_stages: int, is_tail: bool) -> float:
    return float(_lib.stage_clip_threshold(n_stages, 1 if is_tail else 0))


def stage_clip_sumsq(grad: int, count: int, dtype: int, sumsq: int, stream: int = 0) -> None:
    _check(_lib.stage_clip_sumsq(grad or None, count, dtype, sumsq or None, stream or None), "stage_clip_sumsq")


def stage_clip_scale(grad: int, count: int, dtype: int, sumsq: int, threshold: float, stream: int = 0) -> None:
    _check(_lib.stage_clip_scale(grad or None, count, dtype, sumsq or None, threshold, stream or None),
           "stage_clip_scale")
