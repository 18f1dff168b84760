"""The classification the full-size GPU parity tests report (tests/gpu_util.py) on hand-made
cases: which elements over the bound are format-limited, which fell on the wrong side of a
rounding midpoint, which are plain compute errors.  CPU only."""
import numpy as np

from xema_inputs import bf16_bits

from gpu_util import _bf16_neighbours, tolerance_split


def test_bf16_neighbours_and_round_to_nearest_even():
    lo, hi, exact, rne = _bf16_neighbours(np.array([4.009, 8.03, 1.0, 4.015625, 4.046875, -4.009]))
    assert lo.tolist() == [4.0, 8.0, 1.0, 4.0, 4.03125, 4.0]
    assert hi.tolist() == [4.03125, 8.0625, 1.0078125, 4.03125, 4.0625, 4.03125]
    assert exact.tolist() == [False, False, True, False, False, False]
    # 4.015625 and 4.046875 are exact midpoints: ties go to the even mantissa
    assert rne.tolist() == [4.0, 8.0, 1.0, 4.0, 4.0625, 4.0]


def test_tolerance_classes_on_hand_made_elements():
    tol = 0.02
    ref = np.array([4.009, 4.009, 4.009, 8.03, 8.03, 1.0, -4.009, -4.009, 0.5])
    got = np.array([4.0, 4.03125, 4.0625, 8.0, 8.0625, 1.05, -4.03125, 4.03125, 0.5], dtype=np.float32)
    r = tolerance_split(bf16_bits(got), ref, tol)
    # 0: nearest, passes.  1: the far neighbour (error 0.0222 > tol) while the nearest passes.
    # 2: not a neighbour.  3: nearest bf16 of 8.03 is 8.0, error 0.03 > tol: nothing can pass.
    # 4: far neighbour where even the nearest fails: still format-limited.  5: plain error.
    # 6: far neighbour, negative.  7: sign flipped.  8: exact.
    assert r["n"] == 9 and r["n_over"] == 7
    assert r["n_format_limited"] == 2 and [e[0] for e in r["format_limited"]] == [3, 4]
    assert r["n_rounding_side"] == 2 and [e[0] for e in r["rounding_side"]] == [1, 6]
    assert r["n_compute"] == 3
    assert abs(r["max_abs"] - 8.04025) < 1e-9
    i, rf, g, lo, hi, e = r["rounding_side"][1]
    assert (rf, g, lo, hi) == (-4.009, -4.03125, -4.0, -4.03125) and abs(e - 0.02225) < 1e-9
    # with the compute elements removed the remaining maximum is the passing element 0
    keep = np.array([0, 1, 3, 4, 6, 8])
    r2 = tolerance_split(bf16_bits(got[keep]), ref[keep], tol)
    assert r2["n_compute"] == 0 and abs(r2["max_abs_rest"] - 0.009) < 1e-9
    # error minus half a spacing at the reference: 0.02225 - 0.015625 for the far neighbours of 4.009
    assert abs(r2["max_before_rounding"] - 0.006625) < 1e-9
    assert [e[0] for e in r["compute"]] == [2, 5, 7]
