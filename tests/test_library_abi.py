"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

import paper_2002_05814_b200 as hpl
from paper_2002_05814_b200 import build as hpl_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    hpl_build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "hpl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hpl_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"hpl_put", "hpl_reduce", "hpl_broadcast", "hpl_get", "hpl_fail"} <= set(names)
    lib = ctypes.CDLL(hpl.lib_path())
    for n in names:
        assert hasattr(lib, n), n


def test_error_strings_and_argument_checks():
    lib = hpl.load_library()
    for code in range(0, -9, -1):
        assert lib.hpl_strerror(code)
    with pytest.raises(hpl.HplError) as ei:
        hpl.Context(chunk_bytes=24)            # not a multiple of 16
    assert ei.value.code == hpl.HPL_ERR_INVALID
    with hpl.Context(chunk_bytes=64) as c:     # schedule-only context: no device memory given
        c.create(1, 0, 256)
        with pytest.raises(hpl.HplError) as ei:
            c.create(1, 0, 256)
        assert ei.value.code == hpl.HPL_ERR_EXISTS
        with pytest.raises(hpl.HplError) as ei:
            c.create(2, 0, 255)                 # not a whole number of elements
        assert ei.value.code == hpl.HPL_ERR_INVALID
        with pytest.raises(hpl.HplError) as ei:
            c.put(3, 16, 4)
        assert ei.value.code == hpl.HPL_ERR_NOT_FOUND
        with pytest.raises(hpl.HplError) as ei:
            c.put(1, 8, 4)                      # misaligned
        assert ei.value.code == hpl.HPL_ERR_INVALID
        c.put(1, 16, 128)
        with pytest.raises(hpl.HplError) as ei:
            c.put(1, 16, 64)                    # the prefix never shrinks
        assert ei.value.code == hpl.HPL_ERR_INVALID
        with pytest.raises(hpl.HplError) as ei:
            c.advance(5), c.advance(4)
        assert ei.value.code == hpl.HPL_ERR_INVALID
        with pytest.raises(hpl.HplError) as ei:
            c.reduce(9, [1, 1], 1)
        assert ei.value.code == hpl.HPL_ERR_INVALID
        rc, _, _ = c.try_get(1)
        assert rc == hpl.HPL_ERR_TIMEOUT        # partial object
        c.put(1, 16, 256)
        rc, _, _ = c.try_get(1)
        assert rc == hpl.HPL_ERR_CUDA           # complete, but this context has no device
        with pytest.raises(hpl.HplError) as ei:
            c.put_host(1, bytearray(256), 256)
        assert ei.value.code in (hpl.HPL_ERR_CUDA, hpl.HPL_ERR_INVALID)


def test_batch_calls_are_the_single_calls_in_array_order():
    with hpl.Context(chunk_bytes=64) as a, hpl.Context(chunk_bytes=64) as b:
        ids, workers, ptrs = [5, 3, 9, 4], [0, 1, 2, 3], [4096, 8192, 12288, 16384]
        a.create_batch(ids, workers, 256)
        for i, w in zip(ids, workers):
            b.create(i, w, 256)
        a.reduce(100, ids, 3)
        b.reduce(100, ids, 3)
        a.put_batch(ids, ptrs, [256, 128, 256, 64])
        for i, p, n in zip(ids, ptrs, [256, 128, 256, 64]):
            b.put(i, p, n)
        assert a.schedule_dump(100) == b.schedule_dump(100)
        for ctx in (a, b):
            ctx.create(50, 7, 256)
            ctx.create(51, 8, 256)
            ctx.broadcast(5, [50, 51])
        a.join_batch([50, 51], [20480, 24576])
        b.join(50, 20480)
        b.join(51, 24576)
        assert a.schedule_dump(5) == b.schedule_dump(5)
        with pytest.raises(hpl.HplError) as ei:
            a.get_batch([5, 50])                        # object 5 is complete, but there is no device
        assert ei.value.code == hpl.HPL_ERR_CUDA
        with pytest.raises(hpl.HplError) as ei:
            a.create_batch([60, 5], [0, 0], 256)        # the second id exists: the first was still created
        assert ei.value.code == hpl.HPL_ERR_EXISTS
        with pytest.raises(hpl.HplError):
            a.create(60, 0, 256)


def test_the_header_is_plain_c_and_the_library_links_from_c(tmp_path):
    """include/hpl.h compiles as pedantic C99 and a C program linked against the library gets, for the same calls,
    the schedule the Python binding gets."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    libdir = os.path.dirname(hpl.lib_path())
    exe = str(tmp_path / "abi_from_c")
    lib = os.path.basename(hpl.lib_path())[3:-3]                       # libhpl.so -> hpl
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(root, "include"),
                    os.path.join(root, "tests", "abi_from_c.c"), "-L", libdir, "-l" + lib, "-Wl,-rpath," + libdir, "-o", exe],
                   check=True, capture_output=True)
    out = subprocess.run([exe], check=True, capture_output=True, text=True).stdout.splitlines()
    with hpl.Context(chunk_bytes=64) as c:
        for i in (1, 2, 3):
            c.create(i, i - 1, 256)
        c.reduce(9, [1, 2, 3], 2)
        c.advance(10)
        c.put(2, 4096, 256)
        c.advance(20)
        c.put(3, 8192, 128)
        assert [int(x) for x in out[0].split()] == c.schedule_dump(9)
    assert out[1] == lib_strerror(hpl.HPL_ERR_TIMEOUT)


def lib_strerror(code):
    return hpl.load_library().hpl_strerror(code).decode()
