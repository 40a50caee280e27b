"""CPU-side checks of the C ABI: the library loads without a GPU, exports every symbol the
header declares, and its host-only scalar rules agree with the oracle's."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_1806_08342_b200 import build as qbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def qtz():
    qbuild.build()
    from paper_1806_08342_b200 import qtz as q
    q.load_library()
    return q


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "qtz.h")).read()
    return sorted(set(re.findall(r"QTZ_API\s+[\w\s\*]+?\b(qtz_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(qtz):
    lib = qtz.load_library()
    names = declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(qtz.SIGNATURES) == names


def test_status_strings(qtz):
    lib = qtz.load_library()
    assert lib.qtz_status_string(0) == b"ok"
    for code in range(-9, 0):
        assert lib.qtz_status_string(code) not in (b"", b"unknown status")


def test_create_without_gpu_fails_loudly(qtz):
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(qtz.QtzError) as e:
        qtz.Handle(0)
    assert e.value.code == -8


def test_multiplier_matches_oracle(qtz):
    g = np.random.default_rng(0)
    for M in list(10 ** g.uniform(-9, 3, 5000)) + [0.0, 0.5, 1.0, 2.0 ** -31, 1 - 2.0 ** -33, 0.75]:
        assert qtz.quantize_multiplier(float(M)) == oracle.quantize_multiplier(float(M))
    for bad in (-1.0, float("nan"), float("inf"), 2.0 ** 31, 2.0 ** -40):
        with pytest.raises(qtz.QtzError):
            qtz.quantize_multiplier(bad)
        with pytest.raises(oracle.OracleError):
            oracle.quantize_multiplier(bad)


def test_activation_range_and_add_params_match_oracle(qtz):
    g = np.random.default_rng(1)
    for _ in range(2000):
        s = float(np.float32(10 ** g.uniform(-4, 1)))
        z = int(g.integers(0, 256))
        for kind in (0, 1, 2):
            assert qtz.activation_range(kind, s, z) == oracle.activation_range(kind, s, z)
        sa, sb, sy = (float(np.float32(10 ** g.uniform(-3, 0))) for _ in range(3))
        assert qtz.add_params(sa, sb, sy) == oracle.add_params(sa, sb, sy)


def test_params_from_range_matches_oracle(qtz):
    g = np.random.default_rng(2)
    cases = [(2.1, 3.5), (-3.5, -2.1), (0.0, 0.0), (-1.0, 1.0), (0.0, 6.0), (-1e-30, 1e-30)]
    for _ in range(3000):
        lo = float(np.float32(g.normal() * 10 ** g.uniform(-4, 4)))
        cases.append((lo, float(np.float32(lo + abs(g.normal()) * 10 ** g.uniform(-4, 4)))))
    for lo, hi in cases:
        for bits in (4, 8, 16):
            a, b = qtz.params_from_range(lo, hi, bits, False), oracle.affine_params(lo, hi, bits)
            assert a.tobytes() == b.tobytes(), (lo, hi, bits, a, b)
            a, b = qtz.params_from_range(lo, hi, bits, True), oracle.symmetric_params(lo, hi, bits)
            assert a.tobytes() == b.tobytes()


def test_ema_update_matches_oracle_bit_for_bit(qtz):
    g = np.random.default_rng(11)
    n = 7
    lo_a, hi_a, lo_b, hi_b = np.zeros(n), np.zeros(n), np.zeros(n), np.zeros(n)
    init_a = init_b = False
    for step in range(40):
        blo = (g.normal(-1.0, 0.3, n)).astype(np.float32)
        bhi = (g.normal(4.0, 0.5, n)).astype(np.float32)
        decay = [0.9, 0.99, 0.0, 0.5][step % 4]
        init_a = qtz.ema_update(lo_a, hi_a, blo, bhi, decay, init_a)
        init_b = oracle.ema_update(lo_b, hi_b, blo, bhi, decay, init_b)
        assert init_a and init_b
        assert np.array_equal(lo_a.view(np.uint64), lo_b.view(np.uint64))
        assert np.array_equal(hi_a.view(np.uint64), hi_b.view(np.uint64))
    with pytest.raises(qtz.QtzError) as e:
        qtz.ema_update(lo_a, hi_a, np.full(n, np.nan, np.float32), np.ones(n, np.float32), 0.9, True)
    assert e.value.code == -5
    with pytest.raises(qtz.QtzError):
        qtz.ema_update(lo_a, hi_a, np.zeros(n, np.float32), np.ones(n, np.float32), 1.0, True)
    # parameters from the averaged range, same rules on both sides
    for i in range(n):
        a = qtz.params_from_range(np.float32(lo_a[i]), np.float32(hi_a[i]))
        b = oracle.affine_params(np.float32(lo_b[i]), np.float32(hi_b[i]))
        assert a["zero_point"] == b["zero_point"] and a["scale"] == b["scale"]


def test_range_rules_between_layers_match_oracle(qtz):
    g = np.random.default_rng(21)
    for _ in range(2000):
        lo = float(np.float32(g.normal() * 10 ** g.uniform(-3, 2)))
        hi = float(np.float32(lo + abs(g.normal()) * 10 ** g.uniform(-3, 2)))
        for kind in (0, 1, 2):
            assert qtz.range_after_activation(lo, hi, kind) == oracle.range_after_activation(lo, hi, kind)
        pa, pb = oracle.affine_params(lo, hi, 8), oracle.affine_params(-abs(hi), abs(lo) + 1.0, 8)
        for kind in (0, 1, 2):
            assert qtz.add_output_range(pa, pb, kind) == oracle.add_output_range(pa, pb, kind)
    with pytest.raises(qtz.QtzError) as e:
        qtz.range_after_activation(1.0, 0.0, 0)
    assert e.value.code == -1
    with pytest.raises(qtz.QtzError) as e:
        qtz.range_after_activation(float("inf"), 0.0, 0)
    assert e.value.code == -5


def test_accumulator_scales_and_multipliers_match_oracle(qtz):
    g = np.random.default_rng(22)
    wp = np.zeros(300, qtz.QPARAMS)
    wp["scale"] = (10 ** g.uniform(-5, -1, 300)).astype(np.float32)
    for xs, ys in [(np.float32(1 / 255), np.float32(0.0235)), (np.float32(0.047), np.float32(0.013))]:
        acc = qtz.accumulator_scales(xs, wp)
        assert np.array_equal(acc["scale"], xs * wp["scale"]) and not acc["zero_point"].any()
        mult, rshift = qtz.requant_multipliers(xs, wp, ys)
        want = [oracle.quantize_multiplier(float(xs) * float(s) / float(ys)) for s in wp["scale"]]
        assert [(int(m), int(r)) for m, r in zip(mult, rshift)] == want
    for hw in (1, 49, 196, 3136):
        assert qtz.avgpool_multiplier(hw, 0.02, 0.02) == oracle.quantize_multiplier(1.0 / hw)
    assert qtz.avgpool_multiplier(49, np.float32(0.02), np.float32(0.05)) == \
        oracle.quantize_multiplier(float(np.float32(0.02)) / (49.0 * float(np.float32(0.05))))
