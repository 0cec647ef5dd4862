"""CPU-only checks of the boundary: the shared library builds, loads and exports every symbol
that include/adacons.h declares; calls that need a device fail with an error code, not a crash."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2411_03742_b200 import build, binding
    build.build()
    return binding.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "adacons.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adacons_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_four_core_calls():
    names = declared_symbols()
    for core in ("adacons_create", "adacons_aggregate", "adacons_reset", "adacons_destroy"):
        assert core in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_prototypes_cover_the_header(lib):
    for name in declared_symbols():
        fn = getattr(lib, name)
        assert fn.argtypes is not None, f"{name} has no prototype in the binding"


def test_strerror_and_version(lib):
    assert lib.adacons_version() >= 100
    assert lib.adacons_strerror(0) == b"success"
    assert b"unknown" in lib.adacons_strerror(12345)


def test_argument_validation_needs_no_device(lib):
    ctx = ctypes.c_void_p()
    assert lib.adacons_create(None, 4, 10, 0, None, 0) == 1
    assert lib.adacons_create(ctypes.byref(ctx), 0, 10, 0, None, 0) == 1
    assert lib.adacons_create(ctypes.byref(ctx), 4, 10, 9, None, 0) == 1
    assert lib.adacons_destroy(None) == 0
    assert lib.adacons_aggregate(None, None, None, None) == 1
    assert lib.adacons_reset(None, None) == 1


def test_create_without_a_device_returns_an_error_code(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    ctx = ctypes.c_void_p()
    rc = lib.adacons_create(ctypes.byref(ctx), 4, 1024, 0, None, 0)
    assert rc in (4, 5) and not ctx.value


def test_product_does_not_import_the_oracle():
    """The oracle is test infrastructure: nothing in the package may reference it."""
    pkg = os.path.join(ROOT, "paper_2411_03742_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle|oracle[/.]adacons_oracle|#include.*oracle", text, re.M), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2411_03742_b200" not in open(os.path.join(ROOT, "oracle", f)).read(), f


def test_binding_rejects_tensors_that_do_not_match_the_context():
    """The kernels trust their pointers, so the binding checks shape, type, strides and device."""
    import torch
    from paper_2411_03742_b200.binding import check_tensors
    G, out = torch.zeros(4, 100), torch.zeros(100)
    check_tensors(4, 100, "f32", 100, G, out, want_cuda=False)
    for bad_G, bad_out, pitch in [(torch.zeros(4, 99), out, 100), (torch.zeros(5, 100), out, 100),
                                  (G.to(torch.bfloat16), out, 100), (G, torch.zeros(101), 100),
                                  (torch.zeros(100, 4).t(), out, 100), (torch.zeros(4, 200)[:, ::2], out, 100),
                                  (G, torch.zeros(200)[::2], 100), (G, out, 104), (G, out.double(), 100)]:
        with pytest.raises(ValueError):
            check_tensors(4, 100, "f32", pitch, bad_G, bad_out, want_cuda=False)
    padded = torch.zeros(4, 104)[:, :100]
    check_tensors(4, 100, "f32", 104, padded, out, want_cuda=False)          # padded rows are fine
    with pytest.raises(ValueError):
        check_tensors(4, 100, "f32", 100, G, out, want_cuda=True)             # host tensors on the device path


def test_public_header_is_plain_c(tmp_path):
    """include/adacons.h must compile as strict C99 (it is the C ABI) and as C++."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    src = tmp_path / "use_header.c"
    src.write_text('#include "adacons.h"\nint use(void) { adacons_ctx *c = 0; (void)c; return ADACONS_NOALLOC_SCRATCH_BYTES > 0; }\n')
    inc = os.path.join(ROOT, "include")
    for cmd in (["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only"],
                ["g++", "-std=c++17", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c++"]):
        res = subprocess.run(cmd + ["-I", inc, str(src)], capture_output=True, text=True)
        assert res.returncode == 0, res.stderr


def _header_enum(name):
    """{member: value} of `enum name { ... }` in include/adacons.h."""
    text = open(os.path.join(ROOT, "include", "adacons.h")).read()
    body = re.search(r"enum\s+" + name + r"\s*\{(.*?)\};", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    out = {}
    for m in re.finditer(r"(ADACONS_[A-Z0-9_]+)\s*=\s*(0x[0-9a-fA-F]+|\d+)u?", body):
        out[m.group(1)] = int(m.group(2), 0)
    return out


def test_binding_constants_match_the_header():
    """The ctypes binding repeats the header's enumerations as Python constants: every member must be
    there with the header's value (a renumbered option would silently set another one)."""
    from paper_2411_03742_b200 import binding
    for enum, prefix, strip in (("adacons_option", "OPT_", "ADACONS_OPT_"), ("adacons_info", "INFO_", "ADACONS_INFO_"),
                                ("adacons_coeff", "COEFF_", "ADACONS_COEFF_"), ("adacons_flag", "FLAG_", "ADACONS_FLAG_"),
                                ("adacons_error", "", "ADACONS_"), ("adacons_dtype", "", "ADACONS_")):
        members = _header_enum(enum)
        assert members, enum
        for name, value in members.items():
            py = prefix + name[len(strip):]
            assert hasattr(binding, py), f"binding lacks {py} ({name})"
            assert getattr(binding, py) == value, (py, getattr(binding, py), value)
    values = sorted(_header_enum("adacons_option").values())
    assert values == list(range(len(values))), "option keys must be dense: the binding numbers them with range()"


def test_stats_noalloc_binding_validates_before_it_calls(lib):
    """Layout mistakes are caught in Python (ValueError), before any pointer reaches the library."""
    import torch
    from paper_2411_03742_b200 import binding
    G, pq = torch.zeros(4, 64), torch.zeros(8, dtype=torch.float64)
    for bad_G, bad_pq in [(G, pq),                                   # host tensors
                          (G[:, ::2], pq), (G.t(), pq), (G.double(), pq), (torch.zeros(64), pq),
                          (G, pq.float()), (G, torch.zeros(7, dtype=torch.float64)), (G, torch.zeros(16, dtype=torch.float64)[::2])]:
        with pytest.raises(ValueError):
            binding.stats_noalloc(bad_G, bad_pq)
