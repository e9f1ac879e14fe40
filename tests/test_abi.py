"""Host-side checks of the C ABI: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2502_06786_b200 import binding as mq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "matq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(matq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = C.CDLL(mq.lib_path())
    names = _declared()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(mq.EXPORTS)


def test_version_and_strings():
    assert mq.version() >= 100
    assert mq.status_string(mq.OK) == "ok"
    assert "capacity" in mq.status_string(mq.ERR_CAPACITY)
    assert mq.status_string(12345) == "unknown status"


def test_packed_row_bytes():
    assert mq.packed_row_bytes(2304, 8) == 2304
    assert mq.packed_row_bytes(2304, 4) == 1152
    assert mq.packed_row_bytes(2304, 2) == 576
    assert mq.packed_row_bytes(7, 2) == -1 and mq.packed_row_bytes(8, 3) == -1 and mq.packed_row_bytes(0, 4) == -1


def test_argument_errors_are_found_on_the_host():
    lib = mq._lib
    fake = C.c_void_p(0x1000)     # never dereferenced: validation fails first
    null = None
    # quantize
    assert lib.matq_quantize(null, 4, 16, 16, 8, fake, fake, fake, null, null) == mq.ERR_INVALID_ARG
    assert lib.matq_quantize(fake, 4, 16, 8, 8, fake, fake, fake, null, null) == mq.ERR_INVALID_ARG     # ldw < K
    assert lib.matq_quantize(fake, 4, 16, 16, 4, fake, fake, fake, null, null) == mq.ERR_UNSUPPORTED    # c != 8
    # slice_pack
    sp = lib.matq_slice_pack
    assert sp(fake, 4, 16, 8, 0, 0, fake, null, null, null, 0, null, null, null) == mq.ERR_UNSUPPORTED
    assert sp(fake, 4, 16, 8, 9, 0, fake, null, null, null, 0, null, null, null) == mq.ERR_UNSUPPORTED
    assert sp(fake, 4, 16, 8, 3, 0, fake, null, null, null, 0, null, null, null) == mq.ERR_UNSUPPORTED  # r = 3 is not packable
    assert sp(fake, 4, 18, 8, 2, 0, fake, null, null, null, 0, null, null, null) == mq.ERR_SHAPE
    assert sp(fake, 4, 16, 8, 2, 1, fake, null, null, null, 0, null, null, null) == mq.ERR_INVALID_ARG  # E.P. outputs missing
    assert sp(fake, 4, 1 << 17, 8, 2, 1, fake, null, fake, fake, 8, fake, null, null) == mq.ERR_SHAPE   # uint16 columns

    # gemv
    def gemv(packed=fake, N=8, K=128, c=8, r=4, a=fake, z=fake, rp=null, col=null, x=fake, B=1, ldx=128, y=fake, ldy=8, flags=0):
        return lib.matq_gemv(packed, N, K, c, r, a, z, rp, col, x, B, ldx, y, ldy, null, 0, flags, null, null)
    assert gemv(packed=null) == mq.ERR_INVALID_ARG
    assert gemv(B=0) == mq.ERR_INVALID_ARG and gemv(B=17) == mq.ERR_INVALID_ARG
    assert gemv(rp=fake) == mq.ERR_INVALID_ARG                       # overflow pointers come as a pair
    assert gemv(r=3) == mq.ERR_UNSUPPORTED and gemv(c=4) == mq.ERR_UNSUPPORTED
    assert gemv(K=100, ldx=104) == mq.ERR_SHAPE and gemv(ldx=64) == mq.ERR_SHAPE and gemv(ldy=4) == mq.ERR_SHAPE
    assert gemv(packed=C.c_void_p(0x1004)) == mq.ERR_ALIGNMENT
    assert gemv(flags=7) == mq.ERR_INVALID_ARG and gemv(flags=0x200) == mq.ERR_INVALID_ARG
    assert gemv(N=0) == mq.OK                                         # empty problem: nothing to launch


def test_missing_library_fails_loudly(tmp_path):
    # The binding has no fallback: a copy that cannot find libmatq.so beside it must fail at import.
    import importlib.util
    src = os.path.join(ROOT, "paper_2502_06786_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", dst)
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)
