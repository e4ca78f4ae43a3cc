"""The kernels' scalar math, compiled for the host, against libm in fp64 (no GPU).

Checks what the CUDA path relies on: its own Philox matches the published
vectors, and the single-precision screening key stays within the slack that the
kernels allow when they discard indices.  (On the device lg2.approx replaces
log2f; its documented error, 2^-22 relative outside (0.5, 2) and 2^-22 absolute
inside, is added here by hand and checked on the GPU by a test of its own.)
"""
import ctypes as C
import math
import os
import subprocess

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2504_15475_b200", "csrc")


@pytest.fixture(scope="module")
def hm(tmp_path_factory):
    out = str(tmp_path_factory.mktemp("hostmath") / "libersd_math_host.so")
    subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-x", "c++",
                           os.path.join(CSRC, "ersd_math_host.cpp"), "-I", CSRC, "-o", out])
    L = C.CDLL(out)
    L.ersd_host_exact_ln_e.restype = C.c_double
    L.ersd_host_exact_ln_e.argtypes = [C.c_uint32]
    L.ersd_host_exact_key.restype = C.c_double
    L.ersd_host_exact_key.argtypes = [C.c_uint32, C.c_float, C.c_float]
    L.ersd_host_screen_lg2_e.restype = C.c_float
    L.ersd_host_screen_lg2_e.argtypes = [C.c_uint32]
    L.ersd_host_screen_slack.restype = C.c_float
    L.ersd_host_screen_slack.argtypes = [C.c_float]
    L.ersd_host_screen_core.restype = C.c_float
    L.ersd_host_screen_key.restype = C.c_float
    L.ersd_host_screen_key.argtypes = [C.c_uint32, C.c_float, C.c_float]
    L.ersd_host_token_word.restype = C.c_uint32
    L.ersd_host_token_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
    return L


def test_library_philox_matches_published_vectors(hm):
    for line in open(os.path.join(ROOT, "tests", "golden", "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        ctr = (C.c_uint32 * 4)(*w[0:4])
        key = (C.c_uint32 * 2)(*w[4:6])
        out = (C.c_uint32 * 4)()
        hm.ersd_host_philox(ctr, key, out)
        assert list(out) == w[6:10]
    # counter layout (i >> 2, position, sequence, 0), word i & 3, key = (low, high) of the seed
    seed = 0xFEDCBA9876543210
    for i in (0, 5, 6, 7, 100003):
        ctr = (C.c_uint32 * 4)(i >> 2, 11, 22, 0)
        key = (C.c_uint32 * 2)(seed & 0xFFFFFFFF, seed >> 32)
        out = (C.c_uint32 * 4)()
        hm.ersd_host_philox(ctr, key, out)
        assert hm.ersd_host_token_word(seed, 22, 11, i) == out[i & 3]


def test_row_folded_philox_equals_the_plain_one(hm):
    rng = np.random.default_rng(3)
    hm.ersd_host_philox_row.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_void_p]
    for _ in range(300):
        seed = int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2))
        seq, pos, c0 = (int(v) for v in rng.integers(0, 2**32, size=3))
        if _ % 7 == 0:
            seq, pos = 0, 0
        ctr = (C.c_uint32 * 4)(c0, pos, seq, 0)
        key = (C.c_uint32 * 2)(seed & 0xFFFFFFFF, seed >> 32)
        a = (C.c_uint32 * 4)()
        b = (C.c_uint32 * 4)()
        hm.ersd_host_philox(ctr, key, a)
        hm.ersd_host_philox_row(seed, seq, pos, c0, b)
        assert list(a) == list(b)


def _xs():
    rng = np.random.default_rng(0)
    edges = [0, 1, 2, 3, 255, 256, 2**16, 2**23 - 1, 2**23, 2**23 + 1, 2**24, 2**24 + 1,
             2**26 - 1, 2**26, 2**26 + 1,            # w = 2^-6: series / log switch
             2**31 - 1, 2**31, 2**31 + 1, 2**32 - 2**8, 2**32 - 2, 2**32 - 1]
    near = [2**26 + d for d in range(-70, 70)] + [2**31 + d for d in range(-70, 70)]
    logu = (2.0 ** rng.uniform(0, 32, size=200_000)).astype(np.uint64).clip(0, 2**32 - 1)
    uni = rng.integers(0, 2**32, size=200_000, dtype=np.uint64)
    return np.unique(np.concatenate([np.array(edges + near, dtype=np.uint64), logu, uni])).astype(np.uint32)


def test_screening_log_is_within_its_core_bound(hm):
    xs = _xs()
    out = np.empty(xs.shape[0], np.float32)
    hm.ersd_host_screen_lg2_e_many(xs.ctypes.data_as(C.c_void_p), xs.shape[0], out.ctypes.data_as(C.c_void_p))
    w = (xs.astype(np.float64) + 0.5) / 2**32
    true = np.log2(-np.log1p(-w))
    err = np.abs(out.astype(np.float64) - true)
    core = float(hm.ersd_host_screen_core())
    # device-only error of the two lg2.approx: 2^-22 * |value| each, at most 2^-22 * (34 + 1/0.0227)
    device_extra = 2.0**-22 * 80
    assert err.max() + device_extra < core, (err.max(), xs[err.argmax()])
    assert np.isfinite(out).all()


def test_exact_key_matches_libm(hm):
    """The library's own straight-line double-precision ln(-log1p(-w)) against libm, over every
    regime of x (on the host the reciprocal is a plain division; the device's Newton version is
    checked by a GPU test)."""
    worst = 0.0
    for x in _xs()[::7].tolist() + [0, 1, 7, 2**20, 2**31 - 1, 2**31, 2**32 - 1]:
        w = (x + 0.5) / 2**32
        worst = max(worst, abs(hm.ersd_host_exact_ln_e(x) - math.log(-math.log1p(-w))))
    assert worst < 2e-14, worst
    assert hm.ersd_host_exact_key(5, float("nan"), 1.0) == math.inf
    assert hm.ersd_host_exact_key(5, -math.inf, 1.0) == math.inf
    assert hm.ersd_host_exact_key(5, math.inf, 1.0) == -math.inf
    assert hm.ersd_host_exact_key(5, 2.5, 0.0) == -2.5


@pytest.mark.parametrize("T", [0.05, 0.6, 1.0, 4.0])
def test_screening_key_error_is_inside_the_slack(hm, T):
    """|screen key - true key| <= slack(key) / 2 in log2 units, for logits of any plausible size."""
    rng = np.random.default_rng(int(T * 100))
    xs = rng.integers(0, 2**32, size=20_000, dtype=np.uint64)
    xs[:2000] = (2.0 ** rng.uniform(0, 20, size=2000)).astype(np.uint64)
    zs = np.concatenate([rng.normal(size=10_000) * 8, rng.normal(size=5_000) * 300,
                         rng.uniform(-3e4, 3e4, size=5_000)]).astype(np.float32)
    Tf = float(np.float32(T))
    worst = 0.0
    for x, z in zip(xs.tolist(), zs.tolist()):
        a = hm.ersd_host_screen_key(x, z, Tf)
        true = hm.ersd_host_exact_key(x, z, Tf) / math.log(2.0)
        slack = hm.ersd_host_screen_slack(a)
        assert abs(a - true) + 2.0**-22 * 80 <= 0.5 * slack, (x, z, a, true)
        worst = max(worst, abs(a - true) / slack)
    assert worst < 0.5
