"""The C-ABI library loads without a GPU, exports what include/*.h declares, and rejects
host-detectable mistakes before touching the device."""

import ctypes

import pytest


def test_library_exports_every_declared_symbol(libssn):
    names = libssn.declared_symbols()
    assert {"ssn_compress", "ssn_decompress", "ssn_grad_project", "ssn_weight_reproject",
            "ssn_weight_reproject_workspace_bytes", "ssn_status_string", "ssn_version"} <= set(names)
    lib = ctypes.CDLL(libssn.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert libssn.version() >= 100
    assert libssn.status_string(libssn.SSN_OK) == "ok"
    for code in range(1, 6):
        assert libssn.status_string(code) not in ("ok", "unknown status")
    assert libssn.status_string(99) == "unknown status"


def _codec(libssn, **kw):
    args = dict(d=64, k=8, dtype=libssn.SSN_BF16, U=0x1000)
    args.update(kw)
    return libssn.make_codec(**args)


def test_host_validation_needs_no_device(libssn):
    b = libssn
    compress, decompress = b.raw("ssn_compress"), b.raw("ssn_decompress")
    grad, reproj = b.raw("ssn_grad_project"), b.raw("ssn_weight_reproject")
    ok = _codec(b)
    X = Z = 0x2000
    # NULL codec / NULL basis
    assert compress(None, X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_NULL
    assert compress(ctypes.byref(_codec(b, U=0)), X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_NULL
    # impossible ranks and leading dimensions
    assert compress(ctypes.byref(_codec(b, k=65)), X, 64, None, None, 4, 1, Z, 65, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(_codec(b, k=0)), X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(_codec(b, ldu=7)), X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(ok), X, 63, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(ok), X, 64, None, None, 4, 1, Z, 7, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(ok), X, 64, None, None, -1, 1, Z, 8, None, None) == b.SSN_ERR_SHAPE
    assert decompress(ctypes.byref(ok), Z, 8, None, None, 4, 1, X, 10, None, None) == b.SSN_ERR_SHAPE
    # unknown element type
    assert compress(ctypes.byref(_codec(b, dtype=7)), X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_DTYPE
    # missing buffers
    assert compress(ctypes.byref(ok), None, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_NULL
    assert decompress(ctypes.byref(ok), Z, 8, None, None, 4, 1, None, 64, None, None) == b.SSN_ERR_NULL
    # embedding table given but no ids; positional table given but no way to find positions
    withE = _codec(b, E=0x3000, vocab=10)
    assert compress(ctypes.byref(withE), X, 64, None, None, 4, 1, Z, 8, None, None) == b.SSN_ERR_NULL
    withP = _codec(b, P=0x3000, max_pos=10)
    assert compress(ctypes.byref(withP), X, 64, None, None, 4, 0, Z, 8, None, None) == b.SSN_ERR_SHAPE
    assert compress(ctypes.byref(_codec(b, E=0x3000, vocab=10, lde=8)), X, 64, 0x4000, None, 4, 1, Z, 8,
                    None, None) == b.SSN_ERR_SHAPE
    # empty batches are successful no-ops
    assert compress(ctypes.byref(ok), None, 64, None, None, 0, 1, None, 8, None, None) == b.SSN_OK
    assert decompress(ctypes.byref(ok), None, 8, None, None, 0, 1, None, 64, None, None) == b.SSN_OK
    assert grad(ctypes.byref(ok), None, 64, 0, b.SSN_GRAD_COEFF, None, 8, None, 0, None) == b.SSN_OK
    # gradient modes
    assert grad(ctypes.byref(ok), X, 64, 4, 0, Z, 8, None, 0, None) == b.SSN_ERR_DTYPE
    assert grad(ctypes.byref(ok), X, 64, 4, 8, Z, 8, None, 0, None) == b.SSN_ERR_DTYPE
    assert grad(ctypes.byref(ok), X, 64, 4, b.SSN_GRAD_FULL, None, 0, None, 64, None) == b.SSN_ERR_NULL
    assert grad(ctypes.byref(ok), X, 64, 4, b.SSN_GRAD_COEFF, Z, 4, None, 0, None) == b.SSN_ERR_SHAPE
    # re-projection: side, shape containing d, workspace
    ptrs = (ctypes.c_void_p * 1)(0x5000)
    assert reproj(ctypes.byref(ok), ptrs, 1, 32, 64, 64, 5, None, 0, None) == b.SSN_ERR_DTYPE
    assert reproj(ctypes.byref(ok), ptrs, 1, 32, 48, 48, b.SSN_SIDE_RIGHT, None, 0, None) == b.SSN_ERR_SHAPE
    assert reproj(ctypes.byref(ok), ptrs, 1, 32, 64, 64, b.SSN_SIDE_LEFT, None, 0, None) == b.SSN_ERR_SHAPE
    assert reproj(ctypes.byref(ok), ptrs, 1, 32, 64, 60, b.SSN_SIDE_RIGHT, None, 0, None) == b.SSN_ERR_SHAPE
    assert reproj(ctypes.byref(ok), None, 1, 32, 64, 64, b.SSN_SIDE_RIGHT, None, 0, None) == b.SSN_ERR_NULL
    assert reproj(ctypes.byref(ok), ptrs, 0, 32, 64, 64, b.SSN_SIDE_RIGHT, None, 0, None) == b.SSN_OK
    need = b.ssn_weight_reproject_workspace_bytes(ok, 64, 96, b.SSN_SIDE_LEFT, 1)
    assert need > 0
    assert reproj(ctypes.byref(ok), ptrs, 1, 64, 96, 96, b.SSN_SIDE_LEFT, None, 0, None) == b.SSN_ERR_WORKSPACE
    assert reproj(ctypes.byref(ok), ptrs, 1, 64, 96, 96, b.SSN_SIDE_LEFT, 0x6000, need - 1, None) == b.SSN_ERR_WORKSPACE
    nullptrs = (ctypes.c_void_p * 1)(None)
    assert reproj(ctypes.byref(ok), nullptrs, 1, 32, 64, 64, b.SSN_SIDE_RIGHT, None, 0, None) == b.SSN_ERR_NULL


def test_binding_raises_with_a_message(libssn):
    with pytest.raises(libssn.SsnError) as err:
        libssn.ssn_compress(_codec(libssn), 0, 64, 0, 0, 4, 1, 0x2000, 8)
    assert err.value.status == libssn.SSN_ERR_NULL and "NULL" in str(err.value)


def test_validation_from_two_threads_at_once(libssn):
    """Host-side validation touches no shared state: two threads hammering it get the same codes."""
    import threading

    b = libssn
    compress = b.raw("ssn_compress")
    ok, bad = _codec(b), _codec(b, k=65)
    results = [[], []]

    def worker(slot):
        for i in range(2000):
            c = ok if (i + slot) % 2 == 0 else bad
            results[slot].append(compress(ctypes.byref(c), 0x2000, 64, None, None, -1 if c is ok else 4, 1,
                                          0x2000, 65, None, None))

    threads = [threading.Thread(target=worker, args=(s,)) for s in (0, 1)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for slot in (0, 1):
        assert set(results[slot]) == {b.SSN_ERR_SHAPE} and len(results[slot]) == 2000


def test_diagnostics_and_selftest_arguments(libssn):
    b = libssn
    fam, var = b.ssn_last_kernel()
    assert 0 <= fam <= b.SSN_KERNEL_UMMA_TOKENS and var >= 0
    selftest = b.raw("ssn_selftest_bounded_wait")
    assert selftest(1000, None, None) == b.SSN_ERR_NULL
    assert selftest(0, 0x1000, None) == b.SSN_ERR_SHAPE
    assert selftest((1 << 20) + 1, 0x1000, None) == b.SSN_ERR_SHAPE
    # the codec struct carries the optional status word as its last field
    assert b.ssn_codec_t._fields_[-1][0] == "dev_status"
    grad_factor = b.raw("ssn_reparam_grad_factor")
    assert grad_factor(ctypes.byref(_codec(b)), None, 64, 64, None, 64, -1, 0x1000, 8, None, 0, None) == b.SSN_ERR_SHAPE
