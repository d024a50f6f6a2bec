"""Pins of the bf16 step-distance comparison used by the GEMM parity tests (oracle/compare.py)."""
from fractions import Fraction

import numpy as np

from oracle import compare


def test_rounding_to_bf16_is_one_rounding_to_nearest_even():
    # 1 + 2^-8 is the midpoint of 1 and 1 + 2^-7: ties to even -> 1.0 (0x3F80); just above goes up
    cases = {1.0: 0x3F80, 1.0 + 2.0 ** -8: 0x3F80, 1.0 + 2.0 ** -8 + 2.0 ** -40: 0x3F81, 1.0 + 3 * 2.0 ** -8: 0x3F82,
             -(1.0 + 2.0 ** -8): 0xBF80, 0.0: 0x0000, 3.0: 0x4040, 448.0: 0x43E0}
    # a value that rounds to a tie in fp32 first and would then round the wrong way in two steps
    cases[1.0 + 2.0 ** -8 - 2.0 ** -30] = 0x3F80
    cases[1.0 + 2.0 ** -8 + 2.0 ** -30] = 0x3F81
    x = np.array(list(cases.keys()))
    assert compare.bf16_bits_rne(x).tolist() == list(cases.values())


def test_rounding_agrees_with_exact_rational_arithmetic():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-6, 6, 2000),
                        (1.0 + (2 * rng.integers(0, 64, 500) + 1) * 2.0 ** -8) * 2.0 ** rng.integers(-5, 5, 500)])
    got = compare.bf16_bits_rne(x)
    for v, b in zip(x.tolist(), got.tolist()):
        fv = Fraction(v)
        o = int(compare._ordinal(np.array([b], dtype=np.uint16))[0])
        mine = abs(Fraction(float(compare._from_ordinal(np.array([o]))[0])) - fv)
        for nb in (o - 1, o + 1):
            other = abs(Fraction(float(compare._from_ordinal(np.array([nb]))[0])) - fv)
            assert mine < other or (mine == other and o % 2 == 0)


def test_step_report_counts_steps_and_boundaries():
    ref = np.array([1.0, 1.0 + 2.0 ** -8 + 1e-6, 2.0, -3.0, 1.0 + 2.0 ** -9])
    y = np.array([0x3F80, 0x3F80, 0x4001, 0xC040, 0x3F82], dtype=np.uint16)
    rep = compare.bf16_step_report(y, ref, slack=1e-4)
    assert rep["steps"].tolist() == [0, 1, 1, 0, 2]
    # the second value sits 1e-6 from a boundary (allowed to land on either side), the third is a
    # clear miss by one step, the last a clear miss by two
    assert rep["near_mask"].tolist() == [False, True, False, False, False]
    assert rep["off_clear"] == 2 and rep["max_steps"] == 2 and rep["exact"] == 0.4
    # sign of zero does not count as a step
    assert compare.bf16_step_report(np.array([0x8000], dtype=np.uint16), np.array([0.0]), 0.0)["max_steps"] == 0
