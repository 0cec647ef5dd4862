"""The C ABI used from plain C: a C99 program (tests/c_client/adacons_client.c) is compiled with
gcc against include/adacons.h, linked with the shared library and the CUDA runtime, and run on the
hand-worked two-step example (tests/golden/hand_worked_two_steps.txt, exact rationals derived by
hand from Eq. 7, Eq. 11 and Eq. 12-13).  This pins the CUDA path itself -- not only the oracle --
to values that no program produced, and shows that the boundary needs neither Python nor torch."""
import os
import shutil
import subprocess
from fractions import Fraction

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(ROOT, "tests", "golden", "hand_worked_two_steps.txt")
SRC = os.path.join(ROOT, "tests", "c_client", "adacons_client.c")


def _gold():
    vals = {}
    with open(GOLD) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                k, *v = line.split()
                vals[k] = np.array([float(Fraction(t)) for t in v])
    return vals


def _cuda_home():
    for cand in (os.environ.get("CUDA_HOME"), "/usr/local/cuda"):
        if cand and os.path.exists(os.path.join(cand, "include", "cuda_runtime_api.h")):
            return cand
    pytest.skip("CUDA toolkit headers not found")


@pytest.fixture(scope="module")
def client(tmp_path_factory):
    from paper_2411_03742_b200 import binding
    lib = binding.library_path()
    assert os.path.exists(lib), "build the library first"
    gcc = shutil.which("gcc") or pytest.skip("gcc not found")
    cuda = _cuda_home()
    exe = str(tmp_path_factory.mktemp("c_client") / "adacons_client")
    cmd = [gcc, "-std=c99", "-Wall", "-Wextra", "-Werror", "-O1", SRC, "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(cuda, "include"), "-o", exe, lib, "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    return exe


def _run(exe, N, d, beta, steps, values, pitch=None, shards=None):
    args = [exe, str(N), str(d), repr(beta), str(steps)] + ([str(pitch or d)] if pitch or shards else [])
    args += [str(shards)] if shards else []
    res = subprocess.run(args, input=" ".join(repr(float(v)) for v in values), capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stderr
    out = []
    lines = res.stdout.strip().splitlines()
    assert len(lines) == 4 * steps
    for t in range(steps):
        rec = {}
        for line in lines[4 * t:4 * t + 4]:
            k, *v = line.split()
            rec[k] = np.array([float(x) for x in v])
        out.append(rec)
    return out


@pytest.mark.parametrize("pitch", [None, 4], ids=["generic-path", "padded-rows"])
def test_hand_worked_example_through_plain_c(client, pitch):
    """d = 2 fp32 rows are 8 bytes long: contiguous they take the generic kernels; padded to a
    16-byte pitch (the padding is NaN) they take the aligned ones.  Both must give the rationals."""
    g = _gold()
    values = np.concatenate([g["step1.G"], g["step2.G"]])
    got = _run(client, 3, 2, float(g["beta"][0]), 2, values, pitch)
    for t, s in enumerate(("step1", "step2")):
        np.testing.assert_allclose(got[t]["gamma"], g[f"{s}.gamma"], rtol=1e-5, err_msg=f"{s}.gamma")
        np.testing.assert_allclose(got[t]["m"], g[f"{s}.m"], rtol=1e-5, err_msg=f"{s}.m")
        np.testing.assert_allclose(got[t]["out"], g[f"{s}.psi"], rtol=1e-5, err_msg=f"{s}.psi")
        assert got[t]["flags"][0] == 0


def test_collinear_closed_form_through_plain_c(client):
    """Collinear gradients g_i = k_i x: gamma_i = (1/k_i) / sum_j (1/k_j) and out = N / sum_j (1/k_j) * x
    (follows from Eq. 7 and Eq. 12-13; k = (1, 1, 1, 20) damps the outlier to weight 1/61)."""
    rng = np.random.default_rng(11)
    d = 4096
    x = rng.standard_normal(d).astype(np.float32)
    k = np.array([1.0, 1.0, 1.0, 20.0])
    G = (k[:, None] * x[None, :].astype(np.float64)).astype(np.float32)      # rounded to fp32: collinear to 6e-8
    got = _run(client, 4, d, 0.99, 1, G.ravel())[0]
    inv = 1.0 / k
    np.testing.assert_allclose(got["gamma"], inv / inv.sum(), rtol=1e-5)
    np.testing.assert_allclose(got["out"], (4.0 / inv.sum()) * x.astype(np.float64), rtol=1e-5, atol=1e-5 * np.abs(x).max())


def test_hand_worked_example_in_two_halves_through_plain_c(client):
    """The same rationals from the column-sharded form: one context per column of the d = 2 example
    (each a 1-column view of the same device matrix, row pitch 2), adacons_pass1 on both, then
    adacons_finish on both with the two statistics records."""
    g = _gold()
    values = np.concatenate([g["step1.G"], g["step2.G"]])
    got = _run(client, 3, 2, float(g["beta"][0]), 2, values, shards=2)
    for t, s in enumerate(("step1", "step2")):
        np.testing.assert_allclose(got[t]["gamma"], g[f"{s}.gamma"], rtol=1e-5, err_msg=f"{s}.gamma")
        np.testing.assert_allclose(got[t]["m"], g[f"{s}.m"], rtol=1e-5, err_msg=f"{s}.m")
        np.testing.assert_allclose(got[t]["out"], g[f"{s}.psi"], rtol=1e-5, err_msg=f"{s}.psi")
        assert got[t]["flags"][0] == 0


def test_collinear_closed_form_in_three_ranges_through_plain_c(client):
    rng = np.random.default_rng(12)
    d = 4100                                                   # ranges of 1366, 1367, 1367 columns: misaligned views
    x = rng.standard_normal(d).astype(np.float32)
    k = np.array([1.0, 2.0, 4.0, 20.0])
    G = (k[:, None] * x[None, :].astype(np.float64)).astype(np.float32)
    got = _run(client, 4, d, 0.99, 1, G.ravel(), shards=3)[0]
    inv = 1.0 / k
    np.testing.assert_allclose(got["gamma"], inv / inv.sum(), rtol=1e-5)
    np.testing.assert_allclose(got["out"], (4.0 / inv.sum()) * x.astype(np.float64), rtol=1e-5, atol=1e-5 * np.abs(x).max())
