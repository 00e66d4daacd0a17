"""The comparison helpers of the GPU parity tests, checked on the CPU against hand-made faults."""
import numpy as np
import pytest

from oracle import sfb_oracle as orc
from tests.util import C_ROW, assert_lines, worst_line


def test_one_wrong_row_passes_the_frobenius_norm_but_not_the_line_bound():
    rng = np.random.default_rng(3)
    ref = rng.standard_normal((65536, 16))
    got = ref * (1.0 + 1e-4 * rng.standard_normal(ref.shape))        # a healthy result at about 1e-4
    tol = 1e-2
    assert orc.rel_fro(got, ref) <= tol
    assert_lines(got, ref, tol, "healthy")
    bad = got.copy()
    bad[1234] = rng.standard_normal(16)                               # one row replaced by something unrelated
    assert orc.rel_fro(bad, ref) <= tol                              # sqrt(2 / 65536) = 5.5e-3: not seen
    e, r = worst_line(bad, ref, 1)
    assert r == 1234 and e > 0.5
    with pytest.raises(AssertionError, match="row 1234"):
        assert_lines(bad, ref, tol, "one bad row")


def test_a_shifted_strip_of_columns_is_caught():
    rng = np.random.default_rng(4)
    ref = rng.standard_normal((4096, 4096))
    bad = ref.copy()
    bad[128:144, 2048:2080] = ref[128:144, 2016:2048]                 # a 16 x 32 block read from the wrong place
    assert orc.rel_fro(bad, ref) <= 1e-2
    with pytest.raises(AssertionError):
        assert_lines(bad, ref, 1e-2, "shifted block")


def test_rows_that_are_almost_zero_do_not_divide_by_nothing():
    ref = np.zeros((8, 4))
    ref[0] = [3.0, 4.0, 0.0, 0.0]                                     # rms row norm = 5 / sqrt(8)
    got = ref.copy()
    got[5, 0] = 1e-3                                                  # a zero row off by 1e-3 in absolute terms
    e, r = worst_line(got, ref, 1)
    assert r == 5 and e == pytest.approx(1e-3 / (5.0 / np.sqrt(8.0)))
    # an allowance per line (e.g. storage rounding) is taken off the numerator first
    e2, _ = worst_line(got, ref, 1, extra=np.full(8, 1e-3))
    assert e2 == 0.0
    assert C_ROW == 4.0
