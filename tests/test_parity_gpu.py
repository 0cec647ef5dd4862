"""GPU parity: the CUDA library (through its C ABI) against the float64 CPU oracle, element by
element on the same seeded inputs.  Tolerances and the near-tie rule: parity_util.py.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import adacons_oracle as oc
from paper_2411_03742_b200 import workloads as wl
from parity_util import (COEFF_RTOL, OUT_TOL, ULP, assert_coeffs, assert_coeffs_by_set, assert_output, oracle_step,
                         ranks_of, shifted_pass1_applies, streamed_statistics, tally, to_f64, with_kernel_slot_order)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ac():
    from paper_2411_03742_b200 import binding
    binding.load_library()
    return binding


def run_case(ac, w, steps, *, beta=0.99, options=None, oracle_kw=None, offsets=None, per_segment=False,
             fused=False, one_launch=0, expect_path=None, allow_swaps=True, what=None):
    """fused=False keeps small cases on the three-kernel path (the one the large workloads take);
    fused=True lets the library pick the single-pass kernel when the matrix fits in shared memory.
    one_launch: ADACONS_OPT_ONE_LAUNCH (0 = three kernels, 2 = the one-launch kernel whenever possible).
    allow_swaps=False: the recipe's coefficients are well separated, so the kernel's slot order
    must be the oracle's on every step (no near-tie rule)."""
    what = what or w.name
    dev = torch.device("cuda:0")
    oracle_kw = dict(oracle_kw or {})
    h = ac.AdaCons(w.N, w.d, w.dtype, seg_offsets=offsets)
    h.set_option(ac.OPT_FUSED_SMALL, 1 if fused else 0)
    h.set_option(ac.OPT_ONE_LAUNCH, one_launch)
    if per_segment:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
        oracle_kw.update(seg_offsets=offsets, per_segment=True)
        assert h.info(ac.INFO_COEFF_SETS) == len(offsets) - 1
    h.set_option(ac.OPT_BETA, beta)
    for k, v in (options or {}).items():
        h.set_option(k, v)
    orc = oc.AdaConsOracle(w.N, w.d, beta=beta, **oracle_kw)
    out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
    expected_flags = 0
    for t in range(steps):
        G = wl.generate(w, t, dev)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        G64 = to_f64(G)
        res = oracle_step(orc, G64, w.dtype, h.coeffs(ac.COEFF_A), what=what, sort=oracle_kw.get("sort", True),
                          momentum=oracle_kw.get("momentum", True), normalize=oracle_kw.get("normalize", True),
                          allow_swaps=allow_swaps)
        assert_coeffs_by_set(h.coeffs(ac.COEFF_P), res["p"], f"{w.name} step {t} p")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_Q), res["q"], f"{w.name} step {t} q")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_A), res["a"], f"{w.name} step {t} a")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_A_TILDE), res["a_tilde"], f"{w.name} step {t} a~")
        assert_coeffs_by_set(h.coeffs(ac.COEFF_GAMMA), res["gamma"], f"{w.name} step {t} gamma")
        if oracle_kw.get("normalize", True):
            zg, zo = h.normaliser(), res["Z"]
            ok = np.isfinite(zo)
            assert np.all(np.abs(zg[ok] - zo[ok]) <= COEFF_RTOL * np.abs(res["u"][ok]).sum(axis=1) + 1e-300), "Z"
        m, step = h.state()
        assert step == t + 1
        assert_coeffs_by_set(m, res["m"], f"{w.name} step {t} m")
        assert_output(out, res, G64, w.dtype, f"{w.name} step {t}", offsets)
        expected_flags |= int(np.bitwise_or.reduce(res["flags"]))
        assert h.status() == expected_flags
        if expect_path is not None:
            assert h.info(ac.INFO_LAST_PATH) == expect_path
    h.close()
    return h


# ---- the five benchmark configurations, scaled so that the oracle finishes in seconds but the
# ---- kernels still see several tiles per block and a ragged last tile -------------------------
@pytest.mark.parametrize("fused", [False, True])
def test_config1_full_size(ac, fused):
    run_case(ac, wl.WORKLOADS["small4"], 1, fused=fused, expect_path=3 if fused else 1)


@pytest.mark.parametrize("name,d,steps", [
    ("resnet8", 1_000_004, 5),
    ("mixed16", 1_200_008, 4),
    ("bert64", 400_008, 3),
    ("ragged32", 1_000_004, 3),
])
def test_scaled_configs(ac, name, d, steps):
    w = wl.WORKLOADS[name].scaled(d)
    run_case(ac, w, steps, offsets=wl.segment_offsets(w), allow_swaps=(name != "mixed16"))


# ---- each configuration's whole step recipe (50 / 20 / 10 / 100 steps, beta = 0.99) on a shorter
# ---- vector: the momentum state of Eq. 11 is carried through the recipe and compared, with every
# ---- coefficient, the normaliser, the flags and the whole output, on every step ------------------
@pytest.mark.parametrize("name,d,per_segment", [
    ("resnet8", 1_000_004, False),
    ("mixed16", 1_200_008, False),
    ("bert64", 400_008, False),
    ("ragged32", 600_004, False),
    ("ragged32", 600_004, True),
])
def test_full_step_recipe(ac, name, d, per_segment):
    w = wl.WORKLOADS[name].scaled(d)
    run_case(ac, w, w.steps, beta=0.99, offsets=wl.segment_offsets(w), per_segment=per_segment,
             allow_swaps=(name != "mixed16"), what=f"{w.name} recipe" + (" per segment" if per_segment else ""))


@pytest.mark.parametrize("one_launch", [0, 2], ids=["three-kernels", "one-launch"])
def test_config2_full_size_three_steps(ac, one_launch):
    w = wl.WORKLOADS["resnet8"]
    run_case(ac, w, 3, one_launch=one_launch, expect_path=5 if one_launch else 1)


# ---- the one-launch kernel (pass 1, coefficient step by the last block, pass 2) ------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64])
def test_one_launch_all_worker_counts(ac, N, dtype):
    w = wl.Workload(f"ol{N}", N, 200_016, dtype, 3, "gauss", seed=250 + N)
    run_case(ac, w, 3, beta=0.7, one_launch=2, expect_path=5)


@pytest.mark.parametrize("name,d,steps", [("resnet8", 1_000_016, 6), ("mixed16", 1_200_016, 5), ("bert64", 400_016, 4),
                                          ("ragged32", 1_000_008, 4)])
def test_one_launch_scaled_configs(ac, name, d, steps):
    w = wl.WORKLOADS[name].scaled(d)
    run_case(ac, w, steps, one_launch=2, expect_path=5, allow_swaps=(name != "mixed16"), what=f"{w.name} one launch")


def test_one_launch_default_by_size_and_alignment(ac):
    """By default the one-launch kernel serves what does not fit in shared memory, up to 1 GiB, on
    16-byte aligned buffers; per-segment mode keeps the three kernels."""
    dev = torch.device("cuda:0")
    w = wl.Workload("olsel", 8, 2_000_000, "f32", 1, "gauss", seed=2)
    G = wl.generate(w, 0, dev)
    out = torch.empty(w.d + 8, device=dev)
    h = ac.AdaCons(w.N, w.d, "f32")
    assert h.get_option(ac.OPT_ONE_LAUNCH) == 1
    h.aggregate(G, out[:w.d])
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 5 and h.info(ac.INFO_LAUNCHES_PER_CALL) == 1 and h.info(ac.INFO_LAST_PASS2) == 4
    h.aggregate(G, out[4:w.d + 4])                     # out is 16 but not 32 bytes aligned: still one launch
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 5
    h.aggregate(G, out[1:w.d + 1])                     # out is not 16 bytes aligned: fast pass 1, pass 2 with shifted loads
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 1 and h.info(ac.INFO_LAST_PASS2) == 6
    h.set_option(ac.OPT_ONE_LAUNCH, 0)
    h.aggregate(G, out[:w.d])
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 1
    with pytest.raises(ac.AdaConsError):
        h.set_option(ac.OPT_ONE_LAUNCH, 3)
    h2 = ac.AdaCons(w.N, w.d, "f32", seg_offsets=[0, 1000, w.d])
    h2.set_option(ac.OPT_PER_SEGMENT, 1)
    h2.aggregate(G, out[:w.d])
    torch.cuda.synchronize()
    assert h2.info(ac.INFO_LAST_PATH) == 1


@pytest.mark.parametrize("N,d,dtype", [(8, 3_000_000, "f32"), (64, 500_000, "bf16"), (16, 1_500_016, "bf16"), (32, 700_000, "f32")])
def test_one_launch_gives_the_bytes_of_the_three_kernel_path(ac, N, d, dtype):
    """Both paths add the same block partials in the same order and share pass 2's arithmetic: the
    coefficients, the state and the output are bit-identical over several steps with momentum."""
    dev = torch.device("cuda:0")
    w = wl.Workload("olbits", N, d, dtype, 3, "gauss_outlier", seed=N)
    Gs = [wl.generate(w, t, dev) for t in range(3)]
    runs = []
    for mode in (0, 2, 2):
        h = ac.AdaCons(N, d, dtype)
        h.set_option(ac.OPT_FUSED_SMALL, 0)
        h.set_option(ac.OPT_ONE_LAUNCH, mode)
        out = torch.empty(d, dtype=w.torch_dtype, device=dev)
        outs = []
        for G in Gs:
            h.aggregate(G, out)
            outs.append(out.clone())
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == (5 if mode else 1) and h.status() == 0
        runs.append((outs, [h.coeffs(k).copy() for k in range(5)], h.state()[0].copy()))
    for other in runs[1:]:
        for a, b in zip(runs[0][0], other[0]):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
        for a, b in zip(runs[0][1], other[1]):
            assert a.tobytes() == b.tobytes()
        assert runs[0][2].tobytes() == other[2].tobytes()


# ---- every pass-1 instantiation, masked rows, both types ---------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64])
def test_all_worker_counts_fast_path(ac, N, dtype):
    w = wl.Workload(f"n{N}", N, 20_008, dtype, 2, "gauss", seed=50 + N)
    run_case(ac, w, 2, beta=0.7, expect_path=1)


# ---- single-pass kernel (matrix resident in shared memory) --------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 16, 33, 64, 100])
def test_single_pass_kernel_all_worker_counts(ac, N, dtype):
    w = wl.Workload(f"f{N}", N, 20_008, dtype, 3, "gauss", seed=150 + N)
    run_case(ac, w, 3, beta=0.7, fused=True, expect_path=3)


@pytest.mark.parametrize("N,d,dtype", [(4, 4, "f32"), (3, 8, "bf16"), (2, 64 * 4, "f32"), (16, 700_000, "bf16"),
                                       (8, 640_000, "f32")])
def test_single_pass_kernel_sizes(ac, N, d, dtype):
    """One 16-byte vector, exactly one block's worth, and close to the shared-memory capacity."""
    w = wl.Workload(f"fs{N}x{d}", N, d, dtype, 2, "gauss", seed=9)
    run_case(ac, w, 2, beta=0.5, fused=True, expect_path=3)


def test_single_pass_kernel_is_not_used_when_the_matrix_does_not_fit(ac):
    w = wl.Workload("big", 64, 400_008, "bf16", 1, "gauss", seed=1)     # 51 MB > grid shared memory
    run_case(ac, w, 1, fused=True, expect_path=1)


def test_single_pass_and_three_kernel_paths_share_state(ac):
    """Switching between the three paths mid-run continues the same momentum state."""
    w = wl.Workload("mix", 12, 50_000, "f32", 6, "gauss", seed=33)
    dev = "cuda:0"
    h = ac.AdaCons(w.N, w.d, "f32")
    orc = oc.AdaConsOracle(w.N, w.d)
    out = torch.empty(w.d, device=dev)
    for t in range(6):
        h.set_option(ac.OPT_FUSED_SMALL, 1 if t % 3 == 1 else 0)
        h.set_option(ac.OPT_ONE_LAUNCH, 2 if t % 3 == 2 else 0)
        G = wl.generate(w, t, dev)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == (1, 3, 5)[t % 3]
        res = oracle_step(orc, to_f64(G), "f32", h.coeffs(ac.COEFF_A), what="paths share state")
        assert_coeffs(h.coeffs(), res["gamma"], f"gamma step {t}")
        assert_coeffs(h.state()[0], res["m"], f"m step {t}")


def test_path_selection_and_launch_counts(ac):
    w = wl.Workload("probe", 8, 8192, "f32", 1, "gauss")
    h = ac.AdaCons(w.N, w.d, w.dtype)
    G = wl.generate(w, 0, "cuda:0")
    out = torch.empty(w.d, device="cuda:0")
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 3                      # fits in shared memory: one kernel
    assert h.info(ac.INFO_LAUNCHES_PER_CALL) == 1 and h.info(ac.INFO_TOTAL_LAUNCHES) == 1
    h.set_option(ac.OPT_FUSED_SMALL, 0)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 5                      # too large for shared memory by decree: one launch, two reads
    assert h.info(ac.INFO_LAUNCHES_PER_CALL) == 1 and h.info(ac.INFO_TOTAL_LAUNCHES) == 2
    h.set_option(ac.OPT_ONE_LAUNCH, 0)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 1
    assert h.info(ac.INFO_LAUNCHES_PER_CALL) == 3 and h.info(ac.INFO_TOTAL_LAUNCHES) == 5


# ---- generic path: odd lengths, misaligned pointers, many workers ------------------------------
@pytest.mark.parametrize("N,d,dtype", [(4, 10_001, "f32"), (8, 10_003, "bf16"), (3, 2, "f32"), (5, 7, "bf16"),
                                       (65, 5_000, "f32"), (100, 4_099, "bf16"), (128, 3_000, "f32")])
def test_generic_path(ac, N, d, dtype):
    w = wl.Workload(f"g{N}x{d}", N, d, dtype, 2, "gauss", seed=7)
    run_case(ac, w, 2, beta=0.5)


def test_single_column_has_tied_coefficients(ac):
    """d = 1: a_i = sign(g_i) * gbar, so workers of equal sign tie exactly and which of them gets
    which sorted slot depends on rounding.  What is unique: the sorted state, sum(gamma) = 1 and,
    on the first step (where tied slots hold equal values), the output."""
    G = torch.tensor([[0.5], [2.0], [-0.25]], device="cuda:0")
    h, out = _agg(ac, G)
    res = oc.AdaConsOracle(3, 1).step(to_f64(G), storage="f32")
    m, _ = h.state()
    assert_coeffs(np.sort(m[0]), np.sort(res["m"][0]), "sorted state")
    assert abs(h.coeffs().sum() - 1.0) < 1e-12
    assert_output(out, res, to_f64(G), "f32", "d=1")


@pytest.mark.parametrize("aligned_body", [1, 0])
def test_misaligned_base_pointer(ac, aligned_body):
    """A matrix that starts 4 bytes off a 16-byte boundary with a 16-byte pitch: pass 1 runs on the
    aligned body plus the head columns (path 8), or on tensor copies per row class, shifted into place in registers (path 10), when that is switched off;
    `out` is aligned here, i.e. off by another amount than the matrix, so pass 2 shifts its loads into place."""
    N, d = 6, 4096
    w = wl.Workload("mis", N, d, "f32", 1, "gauss", seed=3)
    G0 = wl.generate(w, 0, "cuda:0")
    buf = torch.empty(N * d + 1, device="cuda:0")
    G = buf[1:].view(N, d)
    G.copy_(G0)
    assert G.data_ptr() % 16 != 0
    out = torch.empty(d, device="cuda:0")
    h = ac.AdaCons(N, d, "f32")
    h.set_option(ac.OPT_ALIGNED_BODY, aligned_body)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == (8 if aligned_body else 10) and h.info(ac.INFO_LAST_PASS2) == 6
    res = oc.AdaConsOracle(N, d).step(to_f64(G0), storage="f32")
    assert_coeffs(h.coeffs(ac.COEFF_GAMMA), res["gamma"], "gamma")
    assert_output(out, res, to_f64(G0), "f32", "misaligned")


ALIGNED_BODY_CASES = [  # dtype, N, d, offset of grads (elements), offset of out (elements)
    ("f32", 8, 300_000, 1, 1), ("f32", 8, 300_000, 3, 3), ("f32", 5, 300_000, 2, 0), ("f32", 64, 40_000, 1, 5),
    ("bf16", 16, 400_000, 1, 1), ("bf16", 16, 400_000, 7, 7), ("bf16", 64, 80_000, 5, 13), ("bf16", 3, 400_000, 4, 2),
    ("f32", 4, 8, 1, 1), ("bf16", 4, 16, 3, 3), ("f32", 4, 4, 3, 3), ("bf16", 2, 8, 7, 7),      # hardly any body
    ("f32", 32, 2_000_004, 2, 2), ("bf16", 8, 2_000_008, 6, 6),
]


@pytest.mark.parametrize("dtype,N,d,pitch,off", [("f32", 8, 100_003, 100_008, 1), ("bf16", 24, 77_777, 77_784, 3),
                                                  ("f32", 64, 30_001, 30_004, 2), ("bf16", 5, 9, 16, 5)])
def test_aligned_body_with_padded_rows(ac, dtype, N, d, pitch, off):
    """Both at once: rows padded to a 16-byte pitch (d itself is odd) in a buffer that starts off a
    16-byte boundary, `out` off by the same amount.  NaN in all padding, sentinels around the result."""
    dev = torch.device("cuda:0")
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    w = wl.Workload(f"offpad{N}x{d}", N, d, dtype, 2, "gauss", seed=off + N)
    gbuf = torch.full((N * pitch + 64,), float("nan"), dtype=tdt, device=dev)
    Gp = gbuf[off:off + N * pitch].view(N, pitch)
    obuf = torch.full((d + 64,), 7.0, dtype=tdt, device=dev)
    out = obuf[off:off + d]
    h = ac.AdaCons(N, d, dtype)
    h.set_option(ac.OPT_ROW_PITCH, pitch)
    h.set_option(ac.OPT_BETA, 0.8)
    orc = oc.AdaConsOracle(N, d, beta=0.8)
    for t in range(2):
        G0 = wl.generate(w, t, dev)
        Gp[:, :d] = G0
        h.aggregate(Gp[:, :d], out)
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == 8 and h.info(ac.INFO_LAST_PASS2) == 5
        G64 = to_f64(G0)
        res = oracle_step(orc, G64, dtype, h.coeffs(ac.COEFF_A), what=w.name)
        assert_coeffs(h.coeffs(ac.COEFF_GAMMA)[0], res["gamma"][0], f"{w.name} gamma {t}")
        assert_coeffs(h.state()[0][0], res["m"][0], f"{w.name} m {t}")
        assert_output(out, res, G64, dtype, f"{w.name} out {t}")
        assert bool((obuf[:off] == 7.0).all()) and bool((obuf[off + d:] == 7.0).all()), "wrote outside out"
        assert bool(torch.isnan(Gp[:, d:]).all()) and h.status() == 0
    h.close()


@pytest.mark.parametrize("dtype,N,d,g_off,o_off", ALIGNED_BODY_CASES)
def test_aligned_body_of_offset_buffers(ac, dtype, N, d, g_off, o_off):
    """grads and out are slices of larger buffers that start g_off resp. o_off elements after a
    256-byte boundary; d keeps the row pitch a multiple of 16 bytes.  Pass 1 always takes the aligned
    body; pass 2 does when both are off by the same number of bytes.  NaN before and after the
    matrix, sentinels around the result; three steps with momentum against the oracle."""
    dev = torch.device("cuda:0")
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    eb = 4 if dtype == "f32" else 2
    assert (d * eb) % 16 == 0 and (g_off * eb) % 16 != 0
    w = wl.Workload(f"off{N}x{d}", N, d, dtype, 3, "gauss_outlier", seed=g_off * 16 + o_off)
    gbuf = torch.full((N * d + 64,), float("nan"), dtype=tdt, device=dev)
    G = gbuf[g_off:g_off + N * d].view(N, d)
    obuf = torch.full((d + 64,), 7.0, dtype=tdt, device=dev)
    out = obuf[o_off:o_off + d]
    h = ac.AdaCons(N, d, dtype)
    h.set_option(ac.OPT_BETA, 0.8)
    orc = oc.AdaConsOracle(N, d, beta=0.8)
    same = (g_off * eb) % 16 == (o_off * eb) % 16
    for t in range(3):
        G0 = wl.generate(w, t, dev)
        G.copy_(G0)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        head = (16 - (g_off * eb) % 16) // eb
        assert h.info(ac.INFO_LAST_PATH) == (8 if d > head else 2), h.info(ac.INFO_LAST_PATH)
        assert h.info(ac.INFO_LAST_PASS2) == (5 if same and d > head else 6 if d >= 4 * (16 // eb) else 1)
        G64 = to_f64(G0)
        res = oracle_step(orc, G64, dtype, h.coeffs(ac.COEFF_A), what=w.name)
        for k, code in (("p", ac.COEFF_P), ("q", ac.COEFF_Q), ("a", ac.COEFF_A), ("gamma", ac.COEFF_GAMMA)):
            assert_coeffs(h.coeffs(code)[0], res[k][0], f"{w.name} {k} step {t}")
        assert_coeffs(h.state()[0][0], res["m"][0], f"{w.name} m step {t}")
        assert_output(out, res, G64, dtype, f"{w.name} step {t}")
        assert bool((obuf[:o_off] == 7.0).all()) and bool((obuf[o_off + d:] == 7.0).all()), "wrote outside out"
        assert h.status() == 0
    h.close()


def test_generic_and_fast_paths_agree(ac):
    N, d = 16, 50_000
    w = wl.Workload("agree", N, d, "bf16", 1, "gauss", seed=11)
    G0 = wl.generate(w, 0, "cuda:0")
    buf = torch.empty(N * d + 1, device="cuda:0", dtype=torch.bfloat16)
    G1 = buf[1:].view(N, d)
    G1.copy_(G0)
    o0, o1 = torch.empty(d, device="cuda:0", dtype=torch.bfloat16), torch.empty(d, device="cuda:0", dtype=torch.bfloat16)
    h0, h1 = ac.AdaCons(N, d, "bf16"), ac.AdaCons(N, d, "bf16")
    h0.set_option(ac.OPT_FUSED_SMALL, 0)
    h0.set_option(ac.OPT_ONE_LAUNCH, 0)
    h0.aggregate(G0, o0); h1.aggregate(G1, o1)
    torch.cuda.synchronize()
    assert (h0.info(ac.INFO_LAST_PATH), h1.info(ac.INFO_LAST_PATH)) == (1, 8)
    np.testing.assert_allclose(h0.coeffs(), h1.coeffs(), rtol=2e-6)
    h2, o2 = ac.AdaCons(N, d, "bf16"), torch.empty(d, device="cuda:0", dtype=torch.bfloat16)
    h2.set_option(ac.OPT_ALIGNED_BODY, 0)
    h2.aggregate(G1, o2)
    torch.cuda.synchronize()
    assert h2.info(ac.INFO_LAST_PATH) == 10
    np.testing.assert_allclose(h0.coeffs(), h2.coeffs(), rtol=2e-6)
    np.testing.assert_allclose(to_f64(o1), to_f64(o2), rtol=2e-2, atol=1e-6)
    h3, o3 = ac.AdaCons(N, d, "bf16"), torch.empty(d, device="cuda:0", dtype=torch.bfloat16)
    h3.set_option(ac.OPT_ALIGNED_BODY, 0)
    h3.set_option(ac.OPT_SHIFTED_LOADS, 0)
    h3.aggregate(G1, o3)
    torch.cuda.synchronize()
    assert h3.info(ac.INFO_LAST_PATH) == 2 and h3.info(ac.INFO_LAST_PASS2) == 1
    np.testing.assert_allclose(h0.coeffs(), h3.coeffs(), rtol=2e-6)
    np.testing.assert_allclose(to_f64(o1), to_f64(o3), rtol=2e-2, atol=1e-6)


# ---- per-segment ("layer-wise") coefficients ----------------------------------------------------
def test_per_segment_ragged_layout(ac):
    """390 ragged segments on a 1M-long vector: most tiles hold a segment boundary, many hold several."""
    w = wl.WORKLOADS["ragged32"].scaled(1_000_004)
    run_case(ac, w, 3, beta=0.9, offsets=wl.segment_offsets(w), per_segment=True)


@pytest.mark.parametrize("N,dtype", [(64, "bf16"), (8, "f32"), (16, "bf16"), (3, "f32")])
def test_per_segment_awkward_boundaries(ac, N, dtype):
    """Empty segments, one-column segments, boundaries on and next to tile and vector edges, a
    segment longer than a block's whole tile range."""
    d = 2_400_008
    off = [0, 1, 1, 2, 255, 256, 257, 1024, 1024, 1024, 2048, 2049, 70_000, 70_007, 300_000, 300_000,
           1_900_000, 1_900_001, d - 1, d]
    w = wl.Workload(f"seg{N}", N, d, dtype, 2, "gauss", seed=90 + N)
    run_case(ac, w, 2, beta=0.6, offsets=off, per_segment=True)


def test_per_segment_single_segment_equals_global(ac):
    w = wl.Workload("seg1", 12, 300_000, "f32", 2, "gauss", seed=77)
    dev = "cuda:0"
    h0, h1 = ac.AdaCons(w.N, w.d, "f32"), ac.AdaCons(w.N, w.d, "f32", seg_offsets=[0, w.d])
    h1.set_option(ac.OPT_PER_SEGMENT, 1)
    o0, o1 = torch.empty(w.d, device=dev), torch.empty(w.d, device=dev)
    for t in range(2):
        G = wl.generate(w, t, dev)
        h0.aggregate(G, o0); h1.aggregate(G, o1)
    torch.cuda.synchronize()
    np.testing.assert_allclose(h1.coeffs(), h0.coeffs(), rtol=2e-6)
    np.testing.assert_allclose(to_f64(o1), to_f64(o0), rtol=1e-5, atol=1e-7)


def test_per_segment_needs_the_aligned_path(ac):
    h = ac.AdaCons(4, 1001, "f32", seg_offsets=[0, 500, 1001])
    with pytest.raises(ac.AdaConsError) as e:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
    assert e.value.code == ac.EALIGN
    h = ac.AdaCons(4, 1000, "f32")                      # switching modes resets the state
    G = torch.randn(4, 1000, device="cuda:0")
    out = torch.empty(1000, device="cuda:0")
    h.aggregate(G, out)
    h.set_option(ac.OPT_PER_SEGMENT, 1)
    m, step = h.state()
    assert step == 0 and not m.any()
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.state()[1] == 1


# ---- degenerate inputs --------------------------------------------------------------------------
FUSED_MODE = [0]          # set by the fixture below: the degenerate-input tests run on both paths


@pytest.fixture(params=[0, 1], ids=["three-kernel", "single-pass"])
def both_paths(request):
    FUSED_MODE[0] = request.param
    yield request.param
    FUSED_MODE[0] = 0


def _agg(ac, G, dtype="f32", **opt):
    N, d = G.shape
    h = ac.AdaCons(N, d, dtype)
    h.set_option(ac.OPT_FUSED_SMALL, FUSED_MODE[0])
    for k, v in opt.items():
        h.set_option(k, v)
    out = torch.empty(d, device=G.device, dtype=G.dtype)
    h.aggregate(G, out)
    torch.cuda.synchronize()
    return h, out


def test_identical_gradients_and_single_worker(ac, both_paths):
    g = torch.randn(5000, device="cuda:0")
    h, out = _agg(ac, g.repeat(7, 1).contiguous())
    np.testing.assert_allclose(to_f64(out), to_f64(g), rtol=3e-6, atol=1e-7)
    h, out = _agg(ac, g.view(1, -1).contiguous())
    assert h.coeffs()[0, 0] == 1.0
    assert torch.equal(out, g)


def test_zero_row_all_zero_nonfinite_and_negative_normaliser(ac, both_paths):
    G = torch.randn(4, 4096, device="cuda:0") + torch.randn(4096, device="cuda:0")
    G[2] = 0
    h, out = _agg(ac, G)
    res = oc.AdaConsOracle(4, 4096).step(to_f64(G))
    assert h.status() == ac.FLAG_ZERO_ROW == int(res["flags"][0])
    assert h.coeffs()[0, 2] == 0.0
    assert_coeffs(h.coeffs(), res["gamma"], "gamma zero row")

    h, out = _agg(ac, torch.zeros(3, 1024, device="cuda:0"))
    assert h.status() & ac.FLAG_DEGENERATE_Z and h.status() & ac.FLAG_ZERO_ROW
    np.testing.assert_array_equal(h.coeffs()[0], np.full(3, 1 / 3))
    assert float(out.abs().max()) == 0.0

    G = torch.randn(3, 2048, device="cuda:0") + torch.randn(2048, device="cuda:0")
    h = ac.AdaCons(3, 2048, "f32")
    h.set_option(ac.OPT_FUSED_SMALL, FUSED_MODE[0])
    out = torch.empty(2048, device="cuda:0")
    h.aggregate(G, out)
    m_before, _ = h.state()
    G2 = G.clone(); G2[1, 77] = float("inf")
    h.aggregate(G2, out)
    torch.cuda.synchronize()
    assert h.status() & ac.FLAG_NONFINITE
    np.testing.assert_array_equal(h.coeffs()[0], np.full(3, 1 / 3))
    m_after, step = h.state()
    np.testing.assert_array_equal(m_before, m_after)
    assert step == 2

    x = torch.randn(1024, device="cuda:0")
    h, out = _agg(ac, torch.stack([10 * x, -x]).contiguous())
    assert h.status() & ac.FLAG_NEG_Z
    assert abs(h.coeffs().sum() - 1) < 1e-12


# ---- determinism, state, options ----------------------------------------------------------------
@pytest.mark.parametrize("dtype,d", [("f32", 700_008), ("bf16", 700_008), ("f32", 100_000)])
def test_bit_stability(ac, dtype, d):
    w = wl.Workload("bits", 24, d, dtype, 3, "gauss", seed=21)           # d = 100k: single-pass kernel
    dev = "cuda:0"
    Gs = [wl.generate(w, t, dev) for t in range(3)]
    runs = []
    for _ in range(2):
        h = ac.AdaCons(w.N, w.d, dtype)
        out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
        outs = []
        for G in Gs:
            h.aggregate(G, out)
            outs.append(out.clone())
        torch.cuda.synchronize()
        runs.append((outs, h.coeffs().copy(), h.state()[0].copy()))
    for a, b in zip(runs[0][0], runs[1][0]):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    assert runs[0][1].tobytes() == runs[1][1].tobytes()
    assert runs[0][2].tobytes() == runs[1][2].tobytes()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [100_000, 3_000_008, 1_000_003])
def test_power_of_two_scaling_is_exact(ac, dtype, d):
    """Scaling every gradient by 2^k scales p and q by 4^k, a and m by 2^k and leaves u, Z and gamma
    alone; with a power of two each of these holds without any rounding, so the coefficients must be
    bit-identical and the result must be the scaled result, bit for bit, as long as the squares stay
    in the normal fp32 range.  Covers the single-pass, the TMA and the generic kernels."""
    w = wl.Workload("pow2", 12, d, dtype, 3, "gauss", seed=77)
    dev = "cuda:0"
    Gs = [wl.generate(w, t, dev) for t in range(3)]
    ref = None
    for k in (0, -40, 40):
        h = ac.AdaCons(w.N, w.d, dtype)
        out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
        outs = []
        for G in Gs:
            Gk = (G.float() * 2.0 ** k).to(w.torch_dtype)       # exact: only the exponent changes
            assert torch.equal((Gk.float() * 2.0 ** -k).to(w.torch_dtype), G)
            h.aggregate(Gk, out)
            outs.append((out.float() * 2.0 ** -k).to(w.torch_dtype))
        torch.cuda.synchronize()
        assert h.status() == 0
        got = (outs, h.coeffs(ac.COEFF_GAMMA).copy(), h.coeffs(ac.COEFF_A).copy() * 2.0 ** -k,
               h.state()[0].copy() * 2.0 ** -k, h.coeffs(ac.COEFF_Q).copy() * 4.0 ** -k)
        if ref is None:
            ref = got
            continue
        for a, b in zip(ref[0], got[0]):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), k
        for a, b in zip(ref[1:], got[1:]):
            assert a.tobytes() == b.tobytes(), k


def test_state_roundtrip_and_reset(ac):
    w = wl.Workload("state", 12, 30_000, "f32", 4, "gauss", seed=31)
    dev = "cuda:0"
    h1, h2 = ac.AdaCons(w.N, w.d, "f32"), ac.AdaCons(w.N, w.d, "f32")
    out1, out2 = torch.empty(w.d, device=dev), torch.empty(w.d, device=dev)
    for t in range(2):
        h1.aggregate(wl.generate(w, t, dev), out1)
    m, step = h1.state()
    assert step == 2
    h2.set_state(m, step)
    G = wl.generate(w, 2, dev)
    h1.aggregate(G, out1); h2.aggregate(G, out2)
    torch.cuda.synchronize()
    assert torch.equal(out1, out2) and h2.state()[1] == 3
    h1.reset()
    m, step = h1.state()
    assert step == 0 and not m.any() and h1.status() == 0
    # after a reset the first step is the momentum-free rule
    h1.aggregate(G, out1)
    res = oc.AdaConsOracle(w.N, w.d, beta=0.0).step(to_f64(G))
    assert_coeffs(h1.coeffs(), res["gamma"], "gamma after reset")


@pytest.mark.parametrize("momentum,sorted_,normalize", [(0, 1, 1), (1, 0, 1), (1, 1, 0), (0, 1, 0)])
def test_ablation_variants(ac, momentum, sorted_, normalize):
    w = wl.Workload("abl", 10, 40_000, "f32", 3, "gauss", seed=41)
    run_case(ac, w, 3, beta=0.8,
             options={ac.OPT_MOMENTUM: momentum, ac.OPT_SORTED: sorted_, ac.OPT_NORMALIZE: normalize},
             oracle_kw=dict(momentum=bool(momentum), sort=bool(sorted_), normalize=bool(normalize)))


def test_argument_errors(ac):
    lib = ac.load_library()
    ctx = ctypes.c_void_p()
    assert lib.adacons_create(ctypes.byref(ctx), 0, 10, 0, None, 0) == ac.EINVAL
    assert lib.adacons_create(ctypes.byref(ctx), 4, 0, 0, None, 0) == ac.EINVAL
    assert lib.adacons_create(ctypes.byref(ctx), 4, 10, 7, None, 0) == ac.EINVAL
    assert lib.adacons_create(ctypes.byref(ctx), 2000, 10, 0, None, 0) == ac.EINVAL
    bad = (ctypes.c_int64 * 3)(0, 7, 9)
    assert lib.adacons_create(ctypes.byref(ctx), 4, 10, 0, bad, 2) == ac.EINVAL
    h = ac.AdaCons(4, 1024, "f32")
    G = torch.zeros(4, 1024, device="cuda:0")
    with pytest.raises(ac.AdaConsError):
        h.aggregate_ptr(0, G.data_ptr(), 0)
    with pytest.raises(ac.AdaConsError):
        h.aggregate_ptr(G.data_ptr(), G.data_ptr() + 4096, 0)        # out inside grads
    with pytest.raises(ac.AdaConsError):
        h.set_option(ac.OPT_BETA, 1.5)
    with pytest.raises(ac.AdaConsError):
        h.set_option(99, 1.0)
    assert "invalid" in ac.strerror(ac.EINVAL)


def test_host_entry_point(ac):
    w = wl.Workload("host", 8, 200_000, "bf16", 1, "gauss", seed=61)
    G = wl.generate(w, 0, "cpu").pin_memory()
    out = torch.empty(w.d, dtype=torch.bfloat16).pin_memory()
    h = ac.AdaCons(w.N, w.d, "bf16")
    h.aggregate_host(G, out)
    res = oc.AdaConsOracle(w.N, w.d).step(to_f64(G), storage="bf16")
    assert_coeffs(h.coeffs(), res["gamma"], "gamma host")
    assert_output(out, res, to_f64(G), "bf16", "host entry")


# ---- full size of the large configurations, as the benchmark launches them -----------------------
def full_size_case(ac, name, steps, *, per_segment=False, need_gb=60, allow_swaps=True, sample=200_000):
    """A benchmark configuration at its full size, in the launch configuration bench.py times.
    The oracle's statistics run over ALL columns (streamed through the host in slabs, or one
    segment at a time), so p, q, a, a~, gamma, Z and the state are compared completely on every
    step; the output is compared on sampled columns (both ends, random ones, both sides of every
    segment boundary) against the oracle's combine() with the weights of each column's own set."""
    from concurrent.futures import ThreadPoolExecutor
    w = wl.WORKLOADS[name]
    free, _ = torch.cuda.mem_get_info()
    if free < need_gb * 1e9:
        pytest.skip(f"needs {need_gb} GB of free device memory")
    dev = torch.device("cuda:0")
    off = wl.segment_offsets(w)
    h = ac.AdaCons(w.N, w.d, w.dtype, seg_offsets=off)
    if per_segment:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
    bounds = off if per_segment else [0, w.d]
    S = len(bounds) - 1
    what = f"{name} full size" + (" per segment" if per_segment else "")
    out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
    m = np.zeros((S, w.N))
    gcpu = torch.Generator().manual_seed(1)
    G = None
    for t in range(steps):
        G = wl.generate(w, t, dev, out=G)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == (1 if per_segment or w.N * w.d * w.elem_bytes > 1 << 30 else 5) and h.status() == 0
        if per_segment:
            with ThreadPoolExecutor(max_workers=8) as ex:
                stats = list(ex.map(lambda s_: oc.consensus_statistics(to_f64(G[:, bounds[s_]:bounds[s_ + 1]])), range(S)))
        else:
            stats = [streamed_statistics(G)]
        r_gpu = ranks_of(h.coeffs(ac.COEFF_A))
        want = {k: np.zeros((S, w.N)) for k in ("p", "q", "a", "a_tilde", "gamma", "u")}
        Z = np.zeros(S)
        swapped = 0
        for s_ in range(S):
            c = oc.coefficients(stats[s_][0], stats[s_][1], m[s_], 0.99)          # the oracle alone
            c, n = with_kernel_slot_order(c, r_gpu[s_], what=f"{what} step {t} set {s_}")
            swapped += n
            m[s_] = c["m"]
            Z[s_] = c["Z"]
            for k in want:
                want[k][s_] = c[k]
        tally(what, S, swapped)
        assert allow_swaps or swapped == 0
        for k, code in (("p", ac.COEFF_P), ("q", ac.COEFF_Q), ("a", ac.COEFF_A), ("a_tilde", ac.COEFF_A_TILDE),
                        ("gamma", ac.COEFF_GAMMA)):
            assert_coeffs_by_set(h.coeffs(code), want[k], f"{what} {k} step {t}")
        assert_coeffs_by_set(h.state()[0], m, f"{what} m step {t}")
        assert np.all(np.abs(h.normaliser() - Z) <= COEFF_RTOL * np.abs(want["u"]).sum(axis=1))
        np.testing.assert_allclose(want["gamma"].sum(axis=1), np.ones(S), atol=1e-12)
        if name == "bert64":
            g0 = want["gamma"][0]
            assert g0[0] < 0 and g0[1] < 0 and np.all(g0[2:] > 0)             # the sign-flipped workers
        bnd = torch.tensor(bounds[1:-1], dtype=torch.int64)
        cols = torch.cat([torch.arange(0, 256), torch.arange(w.d - 256, w.d), torch.randint(0, w.d, (sample,), generator=gcpu),
                          bnd - 1, bnd, bnd + 1]).clamp_(0, w.d - 1)
        seg = np.searchsorted(np.asarray(bounds), cols.numpy(), side="right") - 1
        Gs = to_f64(G[:, cols.to(dev)])
        got = to_f64(out[cols.to(dev)])
        psi = np.empty(cols.numel())
        for s_ in np.unique(seg):                                              # the oracle's combine, set by set
            sel = seg == s_
            psi[sel] = oc.combine(Gs[:, sel], want["gamma"][s_])
        gcol = want["gamma"][seg].T
        tight = 1e-5 * np.sum(np.abs(gcol) * np.abs(Gs), axis=0) + ULP[w.dtype] * np.abs(psi) + 1e-45
        assert np.all(np.abs(got - psi) <= tight)
        assert np.all(np.abs(got - psi) <= OUT_TOL[w.dtype] * float(np.abs(Gs).max()) * np.maximum(1.0, np.abs(gcol).sum(axis=0)))
    h.close()


def test_headline_config_full_size(ac):
    """N=64, d=340M, bf16 (43.5 GB), two steps (the second with momentum history)."""
    full_size_case(ac, "bert64", 2)


def test_config5_full_size_model_wise(ac):
    """N=32, d=340M, fp32 (43.5 GB), one set of coefficients for the whole vector, two steps."""
    full_size_case(ac, "ragged32", 2)


def test_config5_full_size_per_segment(ac):
    """The same matrix with layer-wise coefficients: all 390 x 32 coefficients and states."""
    full_size_case(ac, "ragged32", 2, per_segment=True, sample=100_000)


def test_config3_full_size(ac):
    """N=16, d=110M, bf16 (3.5 GB).  Per-worker noise levels spread over two decades keep the
    coefficients far apart: the kernel's slot order must be the oracle's."""
    full_size_case(ac, "mixed16", 2, need_gb=8, allow_swaps=False)


# ---- largest worker counts: the coefficient step's other reduction branch (2N > block size) -----
@pytest.mark.parametrize("N", [512, 600, 1024])
def test_many_workers(ac, N):
    w = wl.Workload(f"many{N}", N, 3_000, "f32", 2, "gauss", seed=N)
    run_case(ac, w, 2, beta=0.9, expect_path=4)
    if N <= 512:
        run_case(ac, w, 2, beta=0.9, options={ac.OPT_CLUSTER_PASS1: 1}, expect_path=6)
    w = wl.Workload(f"manyodd{N}", N, 3_001, "f32", 2, "gauss", seed=N)      # unaligned: generic path
    run_case(ac, w, 2, beta=0.9, expect_path=2)


@pytest.mark.parametrize("N,d,dtype", [(65, 400_008, "bf16"), (100, 300_004, "f32"), (128, 500_000, "bf16"),
                                       (129, 200_000, "bf16"), (200, 150_000, "f32"), (257, 100_008, "bf16"),
                                       (448, 60_000, "bf16"), (512, 50_000, "f32")])
@pytest.mark.parametrize("form", ["default", "clusters", "two-reads"])
def test_more_than_64_workers(ac, N, d, dtype, form):
    """N > 64 on aligned buffers.  Default: up to N = 256 pass 1 reads the matrix once from tiles of
    128 rows x 256 bytes or 256 rows x 128 bytes (rows past N zero-filled); beyond, column sums go to
    scratch and one dot-product launch per 64 rows follows.  Clusters (opt-in): 2, 4 or 8 blocks share each column
    tile, 64 rows per block, the last block's rows ragged or absent."""
    w = wl.Workload(f"big{N}", N, d, dtype, 3, "gauss", seed=N)
    opts = {"default": {}, "clusters": {ac.OPT_CLUSTER_PASS1: 1}, "two-reads": {ac.OPT_TALL_TILES: 0, ac.OPT_CLUSTER_PASS1: 0}}[form]
    path = {"default": 7 if N <= 256 else 4, "clusters": 6, "two-reads": 4}[form]
    run_case(ac, w, 3, beta=0.8, options=opts, expect_path=path)


@pytest.mark.parametrize("N,dtype", [(65, "f32"), (96, "bf16"), (127, "f32"), (128, "bf16"), (128, "f32"),
                                     (129, "bf16"), (200, "f32"), (255, "bf16"), (256, "f32"), (256, "bf16")])
def test_tall_tiles_many_tiles_per_block(ac, N, dtype):
    """The 128- and 256-row tiles on a vector long enough that every block walks many of them (the folding of
    the first-level sums runs several times) with a ragged last tile and heavy-tailed data."""
    w = wl.Workload(f"tall{N}", N, 1_600_008 if N <= 128 else 800_008, dtype, 2, "student_flip", seed=N)
    run_case(ac, w, 2, beta=0.9, expect_path=7)


@pytest.mark.parametrize("N,dtype", [(129, "f32"), (200, "bf16"), (256, "f32"), (256, "bf16")])
def test_tall_tiles_quarter_warp_variant(ac, N, dtype):
    """ADACONS_OPT_TALL_TILES = 2: above 128 workers, tiles of 256 rows x 128 bytes on 256 threads (a
    quarter-warp per row) instead of 256 rows x 256 bytes on 512 threads."""
    w = wl.Workload(f"tallq{N}", N, 800_008, dtype, 2, "student_flip", seed=N + 1)
    run_case(ac, w, 2, beta=0.9, options={ac.OPT_TALL_TILES: 2}, expect_path=7)


@pytest.mark.parametrize("N,dtype", [(128, "f32"), (128, "bf16"), (96, "bf16"), (300, "f32")])
def test_cluster_pass1_many_tiles_per_cluster(ac, N, dtype):
    """Long enough that every cluster walks many tiles (the double-buffered exchange of the partial
    column sums wraps around many times) and the last tile is ragged."""
    w = wl.Workload(f"cl{N}", N, 2_000_008 if N <= 128 else 800_008, dtype, 2, "student_flip", seed=N)
    run_case(ac, w, 2, beta=0.9, options={ac.OPT_CLUSTER_PASS1: 1}, expect_path=6)


@pytest.mark.parametrize("form", ["default", "clusters", "two-reads"])
def test_more_than_64_workers_with_padded_rows(ac, form):
    opts = {"default": {}, "clusters": {ac.OPT_CLUSTER_PASS1: 1}, "two-reads": {ac.OPT_TALL_TILES: 0, ac.OPT_CLUSTER_PASS1: 0}}[form]
    _padded_case(ac, 96, 123_457, "bf16", 123_464, 2, fused=False, options=opts,
                 expect_path={"default": 7, "clusters": 6, "two-reads": 4}[form])


# ---- the call neither allocates nor synchronises: it can be recorded once and replayed -----------
@pytest.mark.parametrize("one_launch", [0, 2], ids=["three-kernels", "one-launch"])
def test_replay_from_a_cuda_graph_advances_the_state(ac, one_launch):
    w = wl.Workload("graph", 16, 600_000, "bf16", 3, "gauss", seed=123)
    dev = torch.device("cuda:0")
    G = wl.generate(w, 0, dev)
    static_G = torch.empty_like(G)
    out = torch.empty(w.d, dtype=torch.bfloat16, device=dev)
    h = ac.AdaCons(w.N, w.d, "bf16")
    h.set_option(ac.OPT_FUSED_SMALL, 0)
    h.set_option(ac.OPT_ONE_LAUNCH, one_launch)
    static_G.copy_(G)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        h.aggregate(static_G, out)                    # warm-up outside the capture (encodes the tensor map)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    h.reset()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        h.aggregate(static_G, out)
    orc = oc.AdaConsOracle(w.N, w.d)
    for t in range(3):
        static_G.copy_(wl.generate(w, t, dev))
        graph.replay()
        torch.cuda.synchronize()
        res = oracle_step(orc, to_f64(static_G), "bf16", h.coeffs(ac.COEFF_A), what="graph replay")
        assert_coeffs(h.coeffs(), res["gamma"], f"gamma replay {t}")
        assert_coeffs(h.state()[0], res["m"], f"m replay {t}")
        assert_output(out, res, to_f64(static_G), "bf16", f"replay {t}")
    assert h.state()[1] == 3 and h.info(ac.INFO_LAST_PATH) == (5 if one_launch else 1) and h.status() == 0


# ---- padded rows: any gradient length on the fast paths ------------------------------------------
def _padded_case(ac, N, d, dtype, pitch, steps, *, fused, options=None, offsets=None, per_segment=False, expect_path=None,
                 expect_pass2=None, out_shift=0, one_launch=0):
    """Rows live in an N x pitch buffer whose padding is NaN; the result buffer is followed by a
    sentinel.  Neither may influence, or be touched by, the aggregation."""
    dev = torch.device("cuda:0")
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    w = wl.Workload(f"pad{N}x{d}", N, d, dtype, steps, "gauss", seed=d % 1000 + N)
    buf = torch.full((N, pitch), float("nan"), dtype=tdt, device=dev)
    obuf = torch.full((out_shift + d + 32,), 7.0, dtype=tdt, device=dev)
    out = obuf[out_shift:out_shift + d]
    h = ac.AdaCons(N, d, dtype, seg_offsets=offsets)
    h.set_option(ac.OPT_ROW_PITCH, pitch)
    h.set_option(ac.OPT_FUSED_SMALL, 1 if fused else 0)
    h.set_option(ac.OPT_ONE_LAUNCH, one_launch)
    oracle_kw = {}
    if per_segment:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
        oracle_kw = dict(seg_offsets=offsets, per_segment=True)
    for k, v in (options or {}).items():
        h.set_option(k, v)
    h.set_option(ac.OPT_BETA, 0.8)
    orc = oc.AdaConsOracle(N, d, beta=0.8, **oracle_kw)
    expected_flags = 0                                 # the status word accumulates until a reset
    for t in range(steps):
        G = wl.generate(w, t, dev)
        buf[:, :d] = G
        h.aggregate(buf[:, :d], out)
        torch.cuda.synchronize()
        if expect_path is not None:
            assert h.info(ac.INFO_LAST_PATH) == expect_path
        if expect_pass2 is not None:
            assert h.info(ac.INFO_LAST_PASS2) == expect_pass2
        G64 = to_f64(G)
        res = oracle_step(orc, G64, dtype, h.coeffs(ac.COEFF_A), what=w.name)
        expected_flags |= int(np.bitwise_or.reduce(res["flags"]))          # an empty segment raises flags
        assert h.status() == expected_flags
        assert_coeffs_by_set(h.coeffs(ac.COEFF_GAMMA), res["gamma"], f"pad gamma {t}")
        assert_coeffs_by_set(h.state()[0], res["m"], f"pad m {t}")
        assert_output(out, res, G64, dtype, f"pad out {t}", offsets)
        assert bool((obuf[out_shift + d:] == 7.0).all()) and bool((obuf[:out_shift] == 7.0).all()), "wrote outside out"
        assert bool(torch.isnan(buf[:, d:]).all())


@pytest.mark.parametrize("N,d,dtype,pitch", [(8, 300_001, "f32", 300_004), (64, 200_003, "bf16", 200_008),
                                             (16, 123_457, "bf16", 123_520), (5, 77_777, "f32", 80_000)])
@pytest.mark.parametrize("fused", [False, True])
def test_padded_rows_odd_length(ac, N, d, dtype, pitch, fused):
    big = N * pitch * (4 if dtype == "f32" else 2) > 20e6
    _padded_case(ac, N, d, dtype, pitch, 2, fused=fused, expect_path=1 if (not fused or big) else 3)


# (dtype, d, pitch, shift of `out` in elements, pass-2 kernel: 2 = 16-byte vectors, 3 = 32-byte vectors)
PASS2_WIDTH_CASES = [
    ("bf16", 200_000, 200_000, 0, 3),    # even number of 16-byte groups, no tail
    ("bf16", 200_003, 200_016, 0, 3),    # odd number of groups, the single last one partial
    ("bf16", 200_011, 200_016, 0, 3),    # even number, the second of the last pair partial
    ("bf16", 200_008, 200_016, 0, 3),    # odd number, full
    ("bf16", 200_008, 200_008, 0, 2),    # pitch is 16 mod 32
    ("bf16", 200_003, 200_008, 0, 2),
    ("bf16", 200_000, 200_000, 8, 2),    # out is 16 mod 32
    ("bf16", 1_000, 1_008, 0, 3),        # less than one block
    ("bf16", 9, 16, 0, 3),               # one pair, second group partial
    ("f32", 100_000, 100_000, 0, 3),
    ("f32", 100_001, 100_008, 0, 3),
    ("f32", 100_006, 100_008, 0, 3),
    ("f32", 100_004, 100_008, 0, 3),
    ("f32", 100_004, 100_004, 0, 2),
    ("f32", 100_002, 100_004, 0, 2),
    ("f32", 100_000, 100_000, 4, 2),
    ("f32", 5, 8, 0, 3),
]


@pytest.mark.parametrize("dtype,d,pitch,shift,kernel", PASS2_WIDTH_CASES)
@pytest.mark.parametrize("N", [3, 8, 13])
def test_pass2_vector_widths(ac, N, dtype, d, pitch, shift, kernel):
    """Pass 2 moves 32 bytes per instruction when grads, out and the pitch are 32-byte aligned and 16
    bytes otherwise; both kernels share one block-to-column mapping.  Every combination of an odd or
    even number of 16-byte groups with a full or partial last group, on both kernels."""
    _padded_case(ac, N, d, dtype, pitch, 2, fused=False, expect_path=1, expect_pass2=kernel, out_shift=shift)


@pytest.mark.parametrize("dtype,d,pitch,shift,kernel", PASS2_WIDTH_CASES)
@pytest.mark.parametrize("N", [3, 13, 40])
def test_one_launch_padded_rows_and_tails(ac, N, dtype, d, pitch, shift, kernel):
    """The one-launch kernel on every tail shape of pass 2 (odd or even number of 16-byte groups,
    full or partial last group, less than one tile, 16- and 32-byte alignment), NaN padding and a
    guarded result."""
    _padded_case(ac, N, d, dtype, pitch, 2, fused=False, one_launch=2, expect_path=5, expect_pass2=4, out_shift=shift)


@pytest.mark.parametrize("dtype,d,pitch,shift,kernel", [c for c in PASS2_WIDTH_CASES if c[1] >= 100_000])
def test_pass2_vector_widths_per_segment(ac, dtype, d, pitch, shift, kernel):
    """The same with one weight set per segment: boundaries inside a 32-byte pair, inside a 16-byte
    group, at block edges, empty and one-column segments."""
    vec = 8 if dtype == "bf16" else 4
    blockc = 512 * vec                                   # columns of one pass-2 block
    top = (d + vec - 1) // vec                           # blocks are counted from the end of the row
    edge = max(0, ((top + 1) // 2 * 2 - 512 * 3)) * vec  # a block edge
    off = sorted({0, 1, 1, vec + 1, 2 * vec, 3 * vec - 1, edge, edge + blockc // 2 + 3, edge + blockc, edge + blockc,
                  d // 2, d // 2 + 1, d - vec - 1, d - 1, d})
    off = [0, 1, 1] + [o for o in off if o > 1 and o < d] + [d - 1, d - 1, d] if d > 4 else [0, d]
    off = sorted(off)
    _padded_case(ac, 11, d, dtype, pitch, 2, fused=False, offsets=off, per_segment=True, expect_path=1,
                 expect_pass2=kernel, out_shift=shift)


def test_padded_rows_per_segment(ac):
    d = 400_003
    off = [0, 3, 100_001, 100_001, 250_000, d - 2, d]
    _padded_case(ac, 12, d, "bf16", 400_008, 2, fused=False, offsets=off, per_segment=True, expect_path=1)


def test_row_pitch_validation_and_unaligned_pitch(ac):
    h = ac.AdaCons(4, 1001, "f32")
    with pytest.raises(ac.AdaConsError):
        h.set_option(ac.OPT_ROW_PITCH, 1000)            # shorter than a row
    # a pitch that is not a multiple of 16 bytes: a tensor map per class of equally offset rows where the classes
    # are thick enough, else the scalar pass 1; pass 2 with shifted loads either way
    _padded_case(ac, 4, 1001, "f32", 1003, 1, fused=True, expect_path=2, expect_pass2=6)
    _padded_case(ac, 16, 1001, "f32", 1003, 1, fused=True, expect_path=10, expect_pass2=6)
    _padded_case(ac, 4, 1001, "bf16", 1003, 1, fused=True, expect_path=10, expect_pass2=6)
    _padded_case(ac, 4, 1001, "bf16", 1003, 1, fused=True, options={ac.OPT_SHIFTED_LOADS: 0}, expect_path=2, expect_pass2=1)


def test_host_entry_point_with_padded_rows(ac):
    N, d, pitch = 6, 50_001, 50_008
    w = wl.Workload("hostpad", N, d, "bf16", 1, "gauss", seed=4)
    G = wl.generate(w, 0, "cpu")
    buf = torch.full((N, pitch), float("nan"), dtype=torch.bfloat16).pin_memory()
    buf[:, :d] = G
    out = torch.empty(d, dtype=torch.bfloat16).pin_memory()
    h = ac.AdaCons(N, d, "bf16")
    h.set_option(ac.OPT_ROW_PITCH, pitch)
    h.aggregate_host(buf[:, :d], out)
    res = oc.AdaConsOracle(N, d).step(to_f64(G), storage="bf16")
    assert_coeffs(h.coeffs(), res["gamma"], "gamma host padded")
    assert_output(out, res, to_f64(G), "bf16", "host padded")


def test_replay_of_the_single_pass_kernel_from_a_cuda_graph(ac):
    """The cooperative single-pass launch can be recorded and replayed as well."""
    w = wl.Workload("graphs", 8, 60_000, "f32", 3, "gauss", seed=321)
    dev = torch.device("cuda:0")
    static_G = wl.generate(w, 0, dev)
    out = torch.empty(w.d, device=dev)
    h = ac.AdaCons(w.N, w.d, "f32")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        h.aggregate(static_G, out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 3
    h.reset()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        h.aggregate(static_G, out)
    orc = oc.AdaConsOracle(w.N, w.d)
    for t in range(3):
        static_G.copy_(wl.generate(w, t, dev))
        graph.replay()
        torch.cuda.synchronize()
        res = oracle_step(orc, to_f64(static_G), "f32", h.coeffs(ac.COEFF_A), what="graph replay single-pass")
        assert_coeffs(h.coeffs(), res["gamma"], f"gamma replay {t}")
        assert_output(out, res, to_f64(static_G), "f32", f"replay {t}")
    assert h.state()[1] == 3 and h.status() == 0


@pytest.mark.parametrize("one_launch", [0, 2], ids=["three-kernels", "one-launch"])
def test_two_contexts_on_two_streams_are_independent(ac, one_launch):
    """Distinct contexts share nothing: interleaved on two streams they give what each gives alone.
    (Two cooperative one-launch kernels cannot share the GPU; the driver runs them one after the
    other, and their waits are on their own contexts' words.)"""
    dev = torch.device("cuda:0")
    wa = wl.Workload("ctxa", 16, 900_008, "bf16", 3, "gauss", seed=1)
    wb = wl.Workload("ctxb", 5, 1_300_000, "f32", 3, "gauss_outlier", seed=2)
    Ga = [wl.generate(wa, t, dev) for t in range(3)]
    Gb = [wl.generate(wb, t, dev) for t in range(3)]

    def alone(w, Gs, dtype):
        h = ac.AdaCons(w.N, w.d, dtype)
        h.set_option(ac.OPT_FUSED_SMALL, 0)
        h.set_option(ac.OPT_ONE_LAUNCH, one_launch)
        out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
        outs = []
        for G in Gs:
            h.aggregate(G, out)
            outs.append(out.clone())
        torch.cuda.synchronize()
        return outs, h.coeffs().copy()

    ref_a, ca = alone(wa, Ga, "bf16")
    ref_b, cb = alone(wb, Gb, "f32")
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    ha, hb = ac.AdaCons(wa.N, wa.d, "bf16"), ac.AdaCons(wb.N, wb.d, "f32")
    ha.set_option(ac.OPT_FUSED_SMALL, 0); hb.set_option(ac.OPT_FUSED_SMALL, 0)
    ha.set_option(ac.OPT_ONE_LAUNCH, one_launch); hb.set_option(ac.OPT_ONE_LAUNCH, one_launch)
    oa = [torch.empty(wa.d, dtype=torch.bfloat16, device=dev) for _ in range(3)]
    ob = [torch.empty(wb.d, device=dev) for _ in range(3)]
    torch.cuda.synchronize()
    for t in range(3):
        ha.aggregate(Ga[t], oa[t], stream=sa)
        hb.aggregate(Gb[t], ob[t], stream=sb)
    torch.cuda.synchronize()
    for t in range(3):
        assert torch.equal(oa[t].view(torch.uint8), ref_a[t].view(torch.uint8))
        assert torch.equal(ob[t], ref_b[t])
    assert ha.coeffs(stream=sa).tobytes() == ca.tobytes() and hb.coeffs(stream=sb).tobytes() == cb.tobytes()
    assert ha.status(stream=sa) == 0 and hb.status(stream=sb) == 0


def test_contexts_of_other_shapes_do_not_disturb_an_existing_one(ac):
    """Contexts whose worker counts fall into the same kernel instantiation (N = 64 and N = 40 share
    the 8 x 8 pass-1 kernel; all N share the generic and the single-pass kernels) need different
    amounts of shared memory.  Creating the smaller plan after the larger one must leave the larger
    one launchable, on every path."""
    dev = torch.device("cuda:0")

    def check(h, w, G):
        out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        res = oc.AdaConsOracle(w.N, w.d).step(to_f64(G)[:, :w.d], storage=w.dtype)
        assert_coeffs(h.coeffs(ac.COEFF_GAMMA), res["gamma"], f"{w.name} gamma")
        assert h.status() == 0

    # TMA-staged pass 1: N = 64 needs more shared memory per stage than N = 40
    big = wl.Workload("shape64", 64, 300_008, "bf16", 1, "gauss", seed=3)
    small = wl.Workload("shape40", 40, 200_000, "bf16", 1, "gauss", seed=4)
    hb = ac.AdaCons(big.N, big.d, "bf16"); hb.set_option(ac.OPT_FUSED_SMALL, 0); hb.set_option(ac.OPT_ONE_LAUNCH, 0)
    hs = ac.AdaCons(small.N, small.d, "bf16"); hs.set_option(ac.OPT_FUSED_SMALL, 0); hs.set_option(ac.OPT_ONE_LAUNCH, 0)
    Gb, Gs = wl.generate(big, 0, dev), wl.generate(small, 0, dev)
    check(hs, small, Gs)
    check(hb, big, Gb)
    assert hb.info(ac.INFO_LAST_PATH) == 1 and hs.info(ac.INFO_LAST_PATH) == 1
    # the allocation-free entry plans a third shape on the same kernel
    pq = torch.empty(2 * 33, dtype=torch.float64, device=dev)
    ac.stats_noalloc(wl.generate(wl.Workload("shape33", 33, 100_000, "bf16", 1, "gauss", seed=5), 0, dev), pq)
    check(hb, big, Gb)
    # generic path (odd length): N = 700 needs 44 KB, N = 3 a few bytes
    gbig = wl.Workload("gen700", 700, 20_001, "f32", 1, "gauss", seed=6)
    gsmall = wl.Workload("gen3", 3, 10_001, "f32", 1, "gauss", seed=7)
    hgb, hgs = ac.AdaCons(gbig.N, gbig.d, "f32"), ac.AdaCons(gsmall.N, gsmall.d, "f32")
    check(hgs, gsmall, wl.generate(gsmall, 0, dev))
    check(hgb, gbig, wl.generate(gbig, 0, dev))
    assert hgb.info(ac.INFO_LAST_PATH) == 2
    # single-pass kernel: a matrix that nearly fills the grid's shared memory, then a tiny one
    fbig = wl.Workload("fused_big", 16, 300_000, "f32", 1, "gauss", seed=8)
    fsmall = wl.Workload("fused_small", 2, 64, "f32", 1, "gauss", seed=9)
    hfb, hfs = ac.AdaCons(fbig.N, fbig.d, "f32"), ac.AdaCons(fsmall.N, fsmall.d, "f32")
    check(hfs, fsmall, wl.generate(fsmall, 0, dev))
    check(hfb, fbig, wl.generate(fbig, 0, dev))
    assert hfb.info(ac.INFO_LAST_PATH) == 3
    for h in (hb, hs, hgb, hgs, hfb, hfs):
        h.close()


def test_profile_and_info_getters(ac):
    w = wl.Workload("prof", 8, 2_000_000, "f32", 1, "gauss", seed=5)
    G = wl.generate(w, 0, "cuda:0")
    out = torch.empty(w.d, device="cuda:0")
    h = ac.AdaCons(w.N, w.d, "f32")
    with pytest.raises(ac.AdaConsError):
        h.profile()                                   # profiling is off
    h.set_option(ac.OPT_PROFILE, 1)
    for _ in range(5):
        h.aggregate(G, out)
    ms, n = h.profile()
    assert n == 5 and all(m > 0 for m in ms) and sum(ms) < 50
    assert h.info(ac.INFO_PASS1_BLOCKS) > 0 and h.info(ac.INFO_SCRATCH_BYTES) > 0
    assert h.info(ac.INFO_NUM_SEGMENTS) == 1 and h.info(ac.INFO_COEFF_SETS) == 1
    assert h.get_option(ac.OPT_BETA) == 0.99 and h.get_option(ac.OPT_ROW_PITCH) == w.d
    with pytest.raises(ac.AdaConsError):
        h.info(99)


def test_vector_longer_than_2_to_the_31(ac):
    """d = 2^31 + 98,760 (N = 2, bf16, 8.6 GB): the TMA coordinates are 32-bit, so pass 1 walks the
    vector in chunks of 2^30 columns.  Statistics from the oracle over all columns; output on
    sampled columns including both sides of every chunk boundary and the very end."""
    N, d = 2, (1 << 31) + 98_760
    free, _ = torch.cuda.mem_get_info()
    if free < 24e9:
        pytest.skip("needs 24 GB of free device memory")
    dev = torch.device("cuda:0")
    w = wl.Workload("long", N, d, "bf16", 1, "gauss", seed=17)
    G = wl.generate(w, 0, dev, row_block=64_000_000)
    out = torch.empty(d, dtype=torch.bfloat16, device=dev)
    h = ac.AdaCons(N, d, "bf16")
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 1 and h.status() == 0
    assert h.info(ac.INFO_LAUNCHES_PER_CALL) == 5                      # three chunks of pass 1
    p, q = streamed_statistics(G, slab=64_000_000, threads=4)
    c = oc.coefficients(p, q, np.zeros(N), 0.99)
    assert_coeffs(h.coeffs(ac.COEFF_P), p, "p")
    assert_coeffs(h.coeffs(ac.COEFF_Q), q, "q")
    assert_coeffs(h.coeffs(ac.COEFF_GAMMA), c["gamma"], "gamma")
    gcpu = torch.Generator().manual_seed(9)
    edges = torch.cat([torch.arange(b - 300, b + 300) for b in (1 << 30, 1 << 31)])
    cols = torch.cat([torch.arange(0, 256), torch.arange(d - 256, d), edges, torch.randint(0, d, (100_000,), generator=gcpu)]).to(dev)
    Gs = to_f64(G[:, cols])
    psi = oc.combine(Gs, c["gamma"])
    got = to_f64(out[cols])
    tight = 1e-5 * (np.abs(c["gamma"])[:, None] * np.abs(Gs)).sum(0) + ULP["bf16"] * np.abs(psi) + 1e-45
    assert np.all(np.abs(got - psi) <= tight)


# ---- seeded random sweep over shapes, types, pitches, segment layouts and paths -------------------
def _random_case(seed):
    r = np.random.default_rng(seed)
    dtype = ["f32", "bf16"][int(r.integers(2))]
    vec = 4 if dtype == "f32" else 8
    N = int(r.choice([1, 2, 3, 5, 8, 9, 16, 17, 31, 32, 33, 48, 64, 65, 70, 130]))
    d = int(r.choice([r.integers(1, 64), r.integers(64, 5_000), r.integers(5_000, 120_000), r.integers(120_000, 400_000)]))
    pad = int(r.choice([0, 0, 1, vec, 3 * vec + 1]))
    pitch = d + pad
    if r.random() < 0.7:                              # most cases: a 16-byte pitch (fast paths)
        pitch = (pitch + vec - 1) // vec * vec
    S = int(r.choice([1, 1, 2, 5, 40]))
    cuts = np.sort(r.integers(0, d + 1, size=S - 1)) if S > 1 else np.array([], dtype=np.int64)
    offsets = [0] + [int(c) for c in cuts] + [d]
    fused = bool(r.random() < 0.5)
    aligned = (pitch * (4 if dtype == "f32" else 2)) % 16 == 0
    per_segment = bool(S > 1 and aligned and N <= 64 and r.random() < 0.7)
    return dict(N=N, d=d, dtype=dtype, pitch=pitch, offsets=offsets, fused=fused, per_segment=per_segment,
                beta=float(r.choice([0.0, 0.5, 0.99])), kind=str(r.choice(["gauss", "gauss_outlier", "student_flip"])))


@pytest.mark.parametrize("seed", range(96))
def test_random_shapes(ac, seed):
    c = _random_case(1000 + seed)
    dev = torch.device("cuda:0")
    tdt = torch.float32 if c["dtype"] == "f32" else torch.bfloat16
    N, d, pitch = c["N"], c["d"], c["pitch"]
    w = wl.Workload(f"rnd{seed}", N, d, c["dtype"], 2, c["kind"], seed=seed)
    buf = torch.full((N, pitch), float("nan"), dtype=tdt, device=dev)
    obuf = torch.full((d + 32,), 7.0, dtype=tdt, device=dev)
    out = obuf[:d]
    h = ac.AdaCons(N, d, c["dtype"], seg_offsets=c["offsets"])
    h.set_option(ac.OPT_ROW_PITCH, pitch)
    h.set_option(ac.OPT_FUSED_SMALL, 1 if c["fused"] else 0)
    h.set_option(ac.OPT_BETA, c["beta"])
    okw = {}
    if c["per_segment"]:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
        okw = dict(seg_offsets=c["offsets"], per_segment=True)
    orc = oc.AdaConsOracle(N, d, beta=c["beta"], **okw)
    flags = 0
    off_ = c["offsets"] if c["per_segment"] else [0, d]
    S = len(off_) - 1
    dm = np.zeros(S)                                   # bound on the error of a set's momentum state
    ulp = ULP[c["dtype"]]
    for t in range(2):
        G = wl.generate(w, t, dev)
        buf[:, :d] = G
        h.aggregate(buf[:, :d], out)
        torch.cuda.synchronize()
        G64 = to_f64(G)
        res = oracle_step(orc, G64, c["dtype"], h.coeffs(ac.COEFF_A), what="random shapes")
        flags |= int(np.bitwise_or.reduce(res["flags"]))
        assert h.status() == flags, c
        # The raw statistics are compared on every set with the bound the arithmetic gives: q_i is a
        # sum of squares (1e-5 relative); p_i = <g_i, gbar> can cancel over a few columns, so its
        # error is measured against cond_i = sum_k |g_ik gbar_k|.  Everything derived from them is
        # compared on every set as well, with those two bounds propagated to first order (times 2):
        #   a_i = p_i/sqrt(q_i)            da_i = 1e-5 (cond_i/sqrt(q_i) + |a_i|)
        #   m   = beta m + (1-beta) S(a)   dm   = beta dm + (1-beta) max_i da_i   (a sort is 1-Lipschitz in max norm)
        #   u_i = a~_i/sqrt(q_i)           du_i = dm/sqrt(q_i) + 1e-5 |u_i|
        #   Z   = sum_i u_i                dZ   = sum_i du_i
        #   gamma_i = u_i/Z                dg_i = (du_i + |gamma_i| dZ)/|Z|
        #   out_k = sum_i gamma_i g_ik     dout_k = sum_i dg_i |g_ik| + one rounding
        # In a well-conditioned set (cond_i ~ |p_i|, |Z| ~ sum|u_i|) these are the 1e-5 relative
        # tolerances of the other tests; a set a few columns wide with sign-flipped workers is
        # allowed the error its own cancellation implies and no more.
        pg, qg, ag, gg = (h.coeffs(k) for k in (ac.COEFF_P, ac.COEFF_Q, ac.COEFF_A, ac.COEFF_GAMMA))
        mg, got = h.state()[0], to_f64(out)
        for s_ in range(S):
            lo, hi = off_[s_], off_[s_ + 1]
            Gs_ = G64[:, lo:hi]
            if hi == lo:
                continue
            cond = np.abs(Gs_) @ np.abs(Gs_.mean(axis=0))
            q_, a_, u_, Z_, gam = res["q"][s_], res["a"][s_], res["u"][s_], res["Z"][s_], res["gamma"][s_]
            assert np.all(np.abs(pg[s_] - res["p"][s_]) <= COEFF_RTOL * cond + 1e-300), f"p set {s_} {c}"
            assert np.all(np.abs(qg[s_] - q_) <= COEFF_RTOL * q_ + 1e-300), f"q set {s_} {c}"
            if int(res["flags"][s_]) & (oc.FLAG_NONFINITE | oc.FLAG_DEGENERATE_Z):
                np.testing.assert_array_equal(gg[s_], gam)        # the documented fallback: exactly 1/N
                continue
            rq = np.where(q_ > 0, np.sqrt(q_), np.inf)            # a zero row has a = u = gamma = 0 exactly
            da = COEFF_RTOL * (cond / rq + np.abs(a_))
            assert np.all(np.abs(ag[s_] - a_) <= 2 * da), f"a set {s_} {c}"
            if np.all(np.abs(res["p"][s_]) >= 1e-2 * cond):       # no cancellation: the plain tolerance
                assert_coeffs(ag[s_], a_, f"a set {s_} {c}")
            dm[s_] = c["beta"] * dm[s_] + (1.0 - c["beta"]) * da.max()
            assert np.all(np.abs(mg[s_] - res["m"][s_]) <= 2 * dm[s_] + 1e-300), f"m set {s_} {c}"
            du = dm[s_] / rq + COEFF_RTOL * np.abs(u_)
            dZ = du.sum()
            if dZ > 0.05 * abs(Z_):                                # the normaliser itself is not determined
                continue
            dg = (du + np.abs(gam) * dZ) / abs(Z_)
            assert np.all(np.abs(gg[s_] - gam) <= 2 * dg), f"gamma set {s_} {c}"
            dout = 2 * (dg @ np.abs(Gs_)) + ulp * np.abs(res["psi"][lo:hi]) + 1e-45
            assert np.all(np.abs(got[lo:hi] - res["psi"][lo:hi]) <= dout), f"out set {s_} {c}"
        assert bool((obuf[d:] == 7.0).all()), "wrote past the end of out"


def test_identical_bf16_gradients_at_scale_are_returned_bit_exactly(ac):
    """64 identical bf16 gradients of 20M elements: every product x*s and x*x has few, structured
    significant bits -- the case in which a single long fp32 sum would drift.  The statistics must
    match the exact sum of squares, the weights must be 1/64, and out must equal g bit for bit."""
    N, d = 64, 20_000_008
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev).manual_seed(4)
    g = (torch.randn(d, generator=gen, device=dev) * 0.01 + 0.003).to(torch.bfloat16)
    G = g.unsqueeze(0).expand(N, d).contiguous()
    out = torch.empty(d, dtype=torch.bfloat16, device=dev)
    h = ac.AdaCons(N, d, "bf16")
    for _ in range(2):                                    # the second step goes through the momentum
        h.aggregate(G, out)
    torch.cuda.synchronize()
    _, q_ref = oc.consensus_statistics(to_f64(g.unsqueeze(0)))
    q, p = h.coeffs(ac.COEFF_Q)[0], h.coeffs(ac.COEFF_P)[0]
    assert np.all(np.abs(q - q_ref[0]) <= 1e-6 * q_ref[0]) and np.all(np.abs(p - q_ref[0]) <= 1e-6 * q_ref[0])
    np.testing.assert_allclose(h.coeffs()[0], np.full(N, 1.0 / N), rtol=1e-12)
    assert torch.equal(out.view(torch.int16), g.view(torch.int16))


# ---- pass 1 from the Gram matrix on the tensor cores (Eq. 7, third line) -----------------------
@pytest.mark.parametrize("fold", [1, 16, 32])
@pytest.mark.parametrize("N,d,recipe", [(64, 700_040, "student_flip"), (48, 300_008, "loguniform"), (33, 150_000, "gauss"),
                                        (16, 400_000, "loguniform"), (5, 90_016, "gauss"), (64, 200, "gauss"), (2, 8, "gauss")])
def test_gram_pass1(ac, N, d, recipe, fold):
    """Row sums and diagonal of the tile Gram matrices against the oracle's statistics; rows past N
    and columns past d come in as zeros; any number of tiles per first-level accumulation."""
    w = wl.Workload(f"gram{N}x{d}", N, d, "bf16", 3, recipe, seed=17 * N + fold)
    run_case(ac, w, 3, options={ac.OPT_GRAM_PASS1: fold}, expect_path=9, what=f"gram{N}")


def test_gram_pass1_many_tiles_per_block(ac):
    """A vector long enough that every block walks its ring many times and folds several times (the
    tensor cores round running sums toward zero: without the second accumulation level q would drift
    out of tolerance as the vector grows)."""
    w = wl.Workload("gram-long", 64, 6_000_008, "bf16", 2, "student_flip", seed=77)
    run_case(ac, w, 2, options={ac.OPT_GRAM_PASS1: 16}, expect_path=9, allow_swaps=False)


def test_gram_pass1_option_is_validated_and_ignored_where_it_does_not_apply(ac):
    h = ac.AdaCons(8, 4096, "f32")
    for bad in (-1, 0.5, 33):
        with pytest.raises(ac.AdaConsError):
            h.set_option(ac.OPT_GRAM_PASS1, bad)
    h.set_option(ac.OPT_GRAM_PASS1, 16)
    h.set_option(ac.OPT_FUSED_SMALL, 0); h.set_option(ac.OPT_ONE_LAUNCH, 0)
    G = torch.randn(8, 4096, device="cuda:0")
    out = torch.empty(4096, device="cuda:0")
    h.aggregate(G, out)
    torch.cuda.synchronize()
    assert h.info(ac.INFO_LAST_PATH) == 1          # fp32 storage: the ordinary kernel
    h.close()


# ---- rows at arbitrary element offsets: 16-byte loads shifted into place ---------------------------
SHIFTED_CASES = [("f32", 8, 100_003, 0, 0), ("f32", 32, 60_001, 0, 0), ("f32", 64, 30_002, 1, 0), ("f32", 17, 44_445, 2, 3), ("f32", 5, 70_001, 1, 2), ("f32", 16, 50_002, 3, 0), ("bf16", 16, 90_001, 0, 0),
                 ("bf16", 7, 65_539, 1, 5), ("bf16", 64, 40_007, 3, 3), ("bf16", 3, 33, 1, 0), ("f32", 3, 16, 0, 1),
                 ("bf16", 100, 30_011, 2, 7), ("f32", 130, 20_001, 1, 1)]


@pytest.mark.parametrize("dtype,N,d,g_off,o_off", SHIFTED_CASES)
def test_rows_at_arbitrary_offsets(ac, dtype, N, d, g_off, o_off):
    """Contiguous rows whose length is not a multiple of 16 bytes: every row starts at another offset
    from a 16-byte boundary, and so may the result.  The vector kernels shift each row's bytes into
    place (pass 1 for N <= 64, pass 2 always); the scalar kernels (option off) must agree.  NaN all around the
    matrix and sentinels around the result: nothing outside is used or touched."""
    dev = torch.device("cuda:0")
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    eb = 4 if dtype == "f32" else 2
    w = wl.Workload(f"shift{N}x{d}", N, d, dtype, 3, "gauss_outlier", seed=7 * g_off + o_off + N)
    gbuf = torch.full((N * d + 64,), float("nan"), dtype=tdt, device=dev)
    G = gbuf[g_off:g_off + N * d].view(N, d)
    obufs = [torch.full((d + 64,), 7.0, dtype=tdt, device=dev) for _ in range(2)]
    outs = [b[o_off:o_off + d] for b in obufs]
    hs = [ac.AdaCons(N, d, dtype) for _ in range(2)]
    hs[1].set_option(ac.OPT_SHIFTED_LOADS, 0)
    for h in hs:
        h.set_option(ac.OPT_BETA, 0.8)
    orc = oc.AdaConsOracle(N, d, beta=0.8)
    for t in range(3):
        G0 = wl.generate(w, t, dev)
        G.copy_(G0)
        for h, o in zip(hs, outs):
            h.aggregate(G, o)
        torch.cuda.synchronize()
        shifted = d >= 4 * (16 // eb)
        assert hs[0].info(ac.INFO_LAST_PASS2) == (6 if shifted else 1) and hs[1].info(ac.INFO_LAST_PASS2) == 1
        if (d * eb) % 16 == 0:                          # rows 16 bytes apart: the staged kernels apply (here only out is off)
            want = 1 if (g_off * eb) % 16 == 0 else 8
            assert hs[0].info(ac.INFO_LAST_PATH) == want and hs[1].info(ac.INFO_LAST_PATH) == want
        else:
            assert hs[0].info(ac.INFO_LAST_PATH) == (10 if shifted_pass1_applies(N, d, dtype) else 2) and hs[1].info(ac.INFO_LAST_PATH) == 2
        G64 = to_f64(G0)
        res = oracle_step(orc, G64, dtype, hs[0].coeffs(ac.COEFF_A), what=w.name)
        for k, code in (("p", ac.COEFF_P), ("q", ac.COEFF_Q), ("a", ac.COEFF_A), ("gamma", ac.COEFF_GAMMA)):
            assert_coeffs(hs[0].coeffs(code)[0], res[k][0], f"{w.name} {k} step {t}")
        assert_coeffs(hs[0].state()[0][0], res["m"][0], f"{w.name} m step {t}")
        assert_output(outs[0], res, G64, dtype, f"{w.name} step {t}")
        if hs[0].info(ac.INFO_LAST_PATH) == hs[1].info(ac.INFO_LAST_PATH):   # the same pass 1, hence the same weights: pass 2 must give the same bytes
            assert torch.equal(outs[0].view(torch.uint8), outs[1].view(torch.uint8))
        else:
            np.testing.assert_allclose(hs[0].coeffs(), hs[1].coeffs(), rtol=4e-6, atol=1e-9)
        for b in obufs:
            assert bool((b[:o_off] == 7.0).all()) and bool((b[o_off + d:] == 7.0).all())
        assert bool(torch.isnan(gbuf[:g_off]).all()) and bool(torch.isnan(gbuf[g_off + N * d:]).all())
        assert hs[0].status() == 0
    for h in hs:
        h.close()


def test_gram_pass1_sums_round_toward_zero(ac):
    """Why the tensor-core pass 1 folds its accumulators: the tensor cores round their running sums
    toward zero, so a sum of squares comes out LOW by an amount that grows with the number of chained
    products (four per tile).  With one tile per fold the error is that of the fp32-pipe kernel; with 32
    it is several 1e-6, still inside the 1e-5 tolerance.  Printed with -s for the record."""
    dev = torch.device("cuda:0")
    N, d = 64, 6_000_008
    w = wl.Workload("gram-rounding", N, d, "bf16", 1, "student_flip", seed=5)
    G = wl.generate(w, 0, dev)
    p_or, q_or = streamed_statistics(G)
    out = torch.empty(d, dtype=torch.bfloat16, device=dev)
    bias = {}
    for fold in (0, 1, 4, 16, 32):
        h = ac.AdaCons(N, d, "bf16")
        h.set_option(ac.OPT_ONE_LAUNCH, 0)
        h.set_option(ac.OPT_GRAM_PASS1, fold)
        h.aggregate(G, out)
        torch.cuda.synchronize()
        assert h.info(ac.INFO_LAST_PATH) == (9 if fold else 1)
        q = h.coeffs(ac.COEFF_Q)[0]
        p = h.coeffs(ac.COEFF_P)[0]
        bias[fold] = float(np.mean((q - q_or) / q_or))
        print(f"tiles per fold {fold:2d}: mean signed rel. error of q {bias[fold]:+.2e}, max |rel. error| of p "
              f"{float(np.max(np.abs(p - p_or) / np.abs(p_or))):.2e}")
        assert np.max(np.abs(q - q_or) / q_or) <= COEFF_RTOL
        h.close()
    assert abs(bias[1]) < 5e-7 and abs(bias[0]) < 5e-7
    assert bias[32] < bias[16] < bias[4] < 0.0 and -1e-5 < bias[32] < -1e-6
