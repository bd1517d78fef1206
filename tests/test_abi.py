"""CPU-side checks of the boundary: the shared library builds, loads without a GPU, exports every
symbol the header declares, and rejects bad arguments on the host before touching a device."""
import ctypes as C
import os
import re
import shutil

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def moqe():
    import paper_2508_09204_b200 as m
    from paper_2508_09204_b200 import build
    if shutil.which("nvcc"):
        build.build()
    return m


def declared_symbols():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"MOQE_API\s+[\w\s\*]+?\b(moqe_\w+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(moqe):
    L = moqe.lib()
    names = declared_symbols()
    assert len(names) >= 16
    for n in names:
        assert hasattr(L, n), f"{n} is declared in include/ but not exported by libmoqe.so"
    assert set(names) == set(moqe.EXPORTED), "binding and header disagree on the entry points"


def test_status_strings(moqe):
    seen = set()
    for code in range(0, 10):
        s = moqe.status_str(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert moqe.status_str(77) == "unknown status"


def test_host_side_argument_checks(moqe):
    L = moqe.lib()
    out = C.c_void_p()
    fake = C.c_void_p(0x1000)          # never dereferenced: the checks below fail first
    assert L.moqe_quantize_rtn(None, 8, 64, 4, 0, 0, None, C.byref(out)) == moqe.ERR_NULL
    assert L.moqe_quantize_rtn(fake, 0, 64, 4, 0, 0, None, C.byref(out)) == moqe.ERR_SHAPE
    assert L.moqe_quantize_rtn(fake, 8, 64, 5, 0, 0, None, C.byref(out)) == moqe.ERR_UNSUPPORTED
    assert L.moqe_quantize_rtn(fake, 8, 60, 4, 0, 0, None, C.byref(out)) == moqe.ERR_UNSUPPORTED
    assert L.moqe_quantize_rtn(fake, 8, 192, 4, 96, 0, None, C.byref(out)) == moqe.ERR_UNSUPPORTED
    assert L.moqe_quantize_rtn(fake, 8, 64, 4, 48, 0, None, C.byref(out)) == moqe.ERR_SHAPE
    assert L.moqe_route(None, 4, 2, fake, None) == moqe.ERR_NULL
    assert L.moqe_route(fake, 4, 0, fake, None) == moqe.ERR_SHAPE
    assert L.moqe_route(fake, 0, 2, fake, None) == moqe.OK
    assert L.moqe_permute(None, fake, 4, 8, 2, None, None, fake, None, 0, None) == moqe.ERR_NULL
    assert L.moqe_permute(None, fake, 4, 8, 33, None, fake, fake, None, 0, None) == moqe.ERR_UNSUPPORTED
    assert L.moqe_permute(fake, fake, 4, 12, 2, fake, fake, fake, None, 0, None) == moqe.ERR_UNSUPPORTED
    assert L.moqe_permute(None, fake, 5000, 8, 2, None, fake, fake, None, 0, None) == moqe.ERR_WORKSPACE
    assert L.moqe_unpermute(fake, fake, -1, 8, fake, None) == moqe.ERR_SHAPE
    assert L.moqe_routed_qgemm(fake, fake, 4, None, 2, fake, fake, 0, None) == moqe.ERR_NULL
    arr = (C.c_void_p * 1)(None)
    assert L.moqe_routed_qgemm(fake, fake, 4, arr, 1, fake, fake, 0, None) == moqe.ERR_NULL
    assert L.moqe_routed_qgemm(fake, fake, 4, arr, 0, fake, fake, 0, None) == moqe.ERR_SHAPE
    assert L.moqe_expert_destroy(None) == moqe.ERR_NULL
    # several layers in one launch: argument checks come before any device work
    xs, ys = (C.c_void_p * 2)(0x1000, 0x2000), (C.c_void_p * 2)(0x3000, 0x4000)
    assert L.moqe_routed_qgemm_sorted_multi(xs, fake, fake, 4, 2, None, 1, ys, fake, 0, None) == moqe.ERR_NULL
    assert L.moqe_routed_qgemm_sorted_multi(xs, fake, fake, 4, 0, arr, 1, ys, fake, 0, None) == moqe.ERR_SHAPE
    assert L.moqe_routed_qgemm_sorted_multi(xs, fake, fake, 4, 17, arr, 2, ys, fake, 0, None) == moqe.ERR_UNSUPPORTED
    assert L.moqe_routed_qgemm_sorted_multi(xs, fake, fake, 4, 1, arr, 1, ys, fake, 0, None) == moqe.ERR_NULL
    assert L.moqe_routed_qgemm_path(fake, fake, 4, arr, 1, fake, fake, 0, None, 6) == moqe.ERR_NULL


def test_workspace_sizes(moqe):
    small = moqe.moqe_routed_qgemm_workspace(16, 4096, 4096, 3)
    big = moqe.moqe_routed_qgemm_workspace(16384, 4096, 4096, 3)
    assert small > 0 and big > 0 and small % 256 == 0 and big % 256 == 0
    assert moqe.moqe_routed_qgemm_workspace(-1, 8, 8, 1) == 0
    assert moqe.lib().moqe_permute_workspace(100, 3) <= moqe.lib().moqe_permute_workspace(100000, 3)


def test_missing_library_fails_loudly(moqe, monkeypatch):
    import paper_2508_09204_b200 as m
    monkeypatch.setattr(m, "_lib", None)
    monkeypatch.setattr(m, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmoqe.so"))
    with pytest.raises(ImportError):
        m.lib()


def test_expert_image_file_errors_without_a_gpu(moqe, tmp_path):
    """A missing file and a file that is not an expert image are refused on the host, before any device call."""
    L = moqe.lib()
    out = C.c_void_p()
    assert L.moqe_expert_host_load(str(tmp_path / "nothing.moqe").encode(), C.byref(out)) == moqe.ERR_IO
    p = tmp_path / "junk.moqe"
    p.write_bytes(b"not an expert image, just forty-eight bytes....!!")
    assert L.moqe_expert_host_load(str(p).encode(), C.byref(out)) == moqe.ERR_UNSUPPORTED
    assert L.moqe_expert_host_load(None, C.byref(out)) == moqe.ERR_NULL
    assert moqe.status_str(moqe.ERR_IO).startswith("file")
