"""The C-ABI library builds, loads on a machine without a GPU, exports every entry point the
header declares, and its host-only functions agree with the oracle.  No device work here."""
import ctypes
import os
import re

import pytest

from oracle import dd_ef_sgd as O
from oracle import deco_policy as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2507_17346_b200 import build
    build.build()
    from paper_2507_17346_b200 import binding
    binding.load()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "deco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(deco_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(B):
    names = declared_functions()
    assert "deco_init" in names and "deco_ef_compress" in names
    assert "deco_aggregate_stale" in names and "deco_apply_update" in names
    assert "deco_set_policy" in names
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), "libdeco.so does not export %s" % name
        assert name in B.SIGNATURES, "binding has no signature for %s" % name
        assert hasattr(B, name), "binding has no wrapper named %s" % name
    assert sorted(B.SIGNATURES) == names


def test_struct_layouts_match_the_header(B):
    assert ctypes.sizeof(B.deco_pair) == 8
    assert ctypes.sizeof(B.deco_lut_entry) == 24
    assert ctypes.sizeof(B.deco_options) == 4 + 4 + 8 + 4 + 4 + 8 + 4 + 4 + 32
    assert ctypes.sizeof(B.deco_stats) == 8 + 8 + 8 + 4 + 4 + 8 + 8 + 8


def test_status_strings(B):
    assert B.status_string(B.DECO_OK) == "ok"
    assert "order" in B.status_string(B.DECO_ERR_STATE)


def test_k_rule_matches_oracle(B):
    for delta, d in [(0.01, 1 << 20), (0.01, 11_689_512), (0.001, 124_439_808),
                     (0.1, 100_000_000), (0.0001, 100_000_000), (0.001, 1_100_048_384),
                     (1.0, 5), (1e-9, 5), (0.3, 10), (0.015625, 100_000_000)]:
        assert B.deco_k_from_delta(delta, d) == O.k_from_delta(delta, d)
    assert B.deco_k_from_delta(0.0, 10) == 0 and B.deco_k_from_delta(1.5, 10) == 0


def test_policy_select_matches_oracle(B):
    import random
    rnd = random.Random(7)
    for _ in range(2000):
        Tc = rnd.uniform(0.01, 0.5)
        b = rnd.uniform(0.0, 0.5)
        a = 10 ** rnd.uniform(7.5, 10.5)
        Vg = 32 * 10 ** rnd.uniform(6, 9)
        non_iid = rnd.random() < 0.3
        tau, delta = B.deco_policy_select(Vg, a, b, Tc, 0, non_iid)
        want = P.deco_select(Vg, a, b, Tc, non_iid)
        assert tau == want[0] and delta == pytest.approx(want[1], rel=1e-12)
        assert B.deco_t_avg(delta, tau, Vg, a, b, Tc) == \
            pytest.approx(P.t_avg(delta, tau, Vg, a, b, Tc), rel=1e-12)
    # tau cap: delta is recomputed for the clamped tau
    tau, delta = B.deco_policy_select(3.2e9, 0.1e9, 0.2, 0.05, 4, False)
    assert tau == 4 and delta == P.delta_star(4, 3.2e9, 0.1e9, 0.2, 0.05)
    with pytest.raises(B.DecoError):
        B.deco_policy_select(0.0, 1e9, 0.1, 0.05)


def test_lut_matches_oracle(B):
    import random
    Vg, b, Tc = 3.2e9, 0.1, 0.05
    lut = B.deco_lut_build(Vg, 0.5e9, 2.0e9, b, Tc, points=20)
    want = P.build_lut(Vg, 0.5e9, 2.0e9, b, Tc, points=20)
    assert len(lut) == 20
    for got, (a, tau, delta) in zip(lut, want):
        assert got.a_bps == pytest.approx(a, rel=1e-15) and got.tau == tau
        assert got.delta == pytest.approx(delta, rel=1e-12)
    rnd = random.Random(3)
    for _ in range(500):
        a = 10 ** rnd.uniform(8.3, 9.6)              # inside and outside [0.5, 2] Gbps
        assert B.deco_lut_lookup(lut, a, Vg, b, Tc) == \
            pytest.approx(P.lut_lookup(want, a, Vg, b, Tc), rel=1e-12)
    one = B.deco_lut_build(Vg, 1e9, 1e9, b, Tc, points=1)
    assert (one[0].tau, one[0].delta) == P.deco_select(Vg, 1e9, b, Tc)
    with pytest.raises(B.DecoError):
        B.deco_lut_build(Vg, 2e9, 1e9, b, Tc, points=5)


def test_init_without_a_device_fails_loudly(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(B.DecoError) as err:
        B.deco_init(1024, 2, 0.1, 1, 0.1)
    assert err.value.status == B.DECO_ERR_CUDA


def test_argument_errors_need_no_device(B):
    lib = B.load()
    ctx = ctypes.c_void_p()
    assert lib.deco_init(None, 10, 1, 0.1, 0, 0.1, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_init(ctypes.byref(ctx), 0, 1, 0.1, 0, 0.1, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_init(ctypes.byref(ctx), 10, 0, 0.1, 0, 0.1, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_init(ctypes.byref(ctx), 10, 1, 0.0, 0, 0.1, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_init(ctypes.byref(ctx), 10, 1, 1.5, 0, 0.1, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_ef_compress(None, None, None) == B.DECO_ERR_INVALID_ARG
    assert lib.deco_get_k(None, None) == B.DECO_ERR_INVALID_ARG
    lib.deco_destroy(None)
