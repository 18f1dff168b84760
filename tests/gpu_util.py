"""Helpers for the GPU parity tests: device upload of bf16 bit patterns and error statistics."""
import numpy as np
import torch

from xema_inputs import bf16_bits, bits_to_f64

DEV = "cuda:0"


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV)


def from_dev_bf16(t: torch.Tensor) -> np.ndarray:
    """int16-viewed bf16 device tensor -> float64 numpy."""
    return bits_to_f64(t.cpu().numpy().view(np.uint16))


def rand_bf16(rng, shape, scale=1.0):
    """(uint16 bits, exact float64 values) of N(0, scale^2) rounded to bf16."""
    bits = bf16_bits((rng.standard_normal(shape, dtype=np.float32) * np.float32(scale)))
    return bits, bits_to_f64(bits)


def stats(got: np.ndarray, ref: np.ndarray) -> dict:
    got = np.asarray(got, np.float64).ravel()
    ref = np.asarray(ref, np.float64).ravel()
    rms = float(np.sqrt(np.mean(ref * ref)))
    err = np.abs(got - ref)
    cos = float(got @ ref / (np.linalg.norm(got) * np.linalg.norm(ref) + 1e-300))
    return {"max_abs": float(err.max()), "rms_ref": rms, "rel": float(err.max() / (rms + 1e-300)), "cos": cos,
            "finite": bool(np.isfinite(got).all())}


def assert_close(got, ref, what, rel=2e-2, cos=0.9995):
    """max-abs error <= rel * RMS(ref) and cosine >= cos."""
    s = stats(got, ref)
    assert s["finite"], (what, "non-finite output")
    assert s["rel"] <= rel and s["cos"] >= cos, (what, s)
    return s


def assert_bf16_close(got, ref, what, atol_rms=2e-3, cos=0.99999):
    """Element-wise bound for a bf16-rounded result: |got - ref| <= 2^-8 |ref| (half an ulp,
    with 15 % slack) + atol_rms * RMS(ref) for the fp32 arithmetic in front of the rounding."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    s = stats(got, ref)
    assert s["finite"], (what, "non-finite output")
    bound = 1.15 * 2.0 ** -8 * np.abs(ref) + atol_rms * s["rms_ref"]
    excess = np.abs(got - ref) - bound
    assert excess.max() <= 0 and s["cos"] >= cos, (what, s, float(excess.max()))
    return s


def _bf16_neighbours(ref: np.ndarray):
    """(lo, hi, exact, rne): magnitudes of the two bf16 numbers bracketing |ref| (fp32 view of the
    float64 reference), whether |ref| is itself a bf16 number, and |ref| rounded to nearest-even."""
    r32 = ref.astype(np.float32)
    mag = r32.view(np.uint32) & np.uint32(0x7FFFFFFF)
    lo_bits = mag & np.uint32(0xFFFF0000)
    lo = lo_bits.view(np.float32).astype(np.float64)
    hi = (lo_bits + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    exact = (mag & np.uint32(0xFFFF)) == 0
    rne_bits = (mag + np.uint32(0x7FFF) + ((mag >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    rne = rne_bits.view(np.float32).astype(np.float64)
    return lo, hi, exact, rne


def tolerance_split(got_bits: np.ndarray, ref: np.ndarray, tol: float, list_max: int = 16) -> dict:
    """Classifies the elements whose error exceeds `tol` into three disjoint classes.

    format_limited   |bf16_rne(ref) - ref| > tol: the exactly rounded reference itself misses
                     the bound (possible where half a bf16 spacing exceeds tol, |y| >= 8 for
                     tol = 2e-2 * RMS with RMS ~ 1.1).  No bf16 output can pass there.
    rounding_side    the correctly rounded reference would pass, and the GPU value is the OTHER
                     of the two bf16 numbers bracketing the reference (a faithful rounding that
                     fell on the far side of a rounding midpoint; needs a spacing > tol, i.e.
                     |y| >= 4).  These break the stated bound and are counted and listed as
                     such; they are not excused.
    compute          everything else over the tolerance: the GPU value is not even a neighbour
                     of the reference.
    Also returned: the raw max-abs; the max-abs over elements outside the first two classes;
    `max_before_rounding` = max(|error| - half a bf16 spacing at the reference), a lower bound
    on the error the value carried before its final rounding to bf16; and the first `list_max`
    elements of every class as (flat index, reference, gpu value, lower neighbour, upper
    neighbour, error)."""
    got = bits_to_f64(got_bits).ravel()
    ref = np.asarray(ref, np.float64).ravel()
    err = np.abs(got - ref)
    over = err > tol
    lo, hi, exact, rne = _bf16_neighbours(ref)
    g = np.abs(got)
    same_sign = (np.signbit(got) == np.signbit(ref)) | (got == 0)
    faithful = same_sign & ((g == lo) | ((g == hi) & ~exact))
    fmt = over & (np.abs(rne - np.abs(ref)) > tol)
    side = over & ~fmt & faithful
    comp = over & ~fmt & ~side
    rest = np.where(fmt | side, 0.0, err)
    before = err - 0.5 * (hi - lo)

    def listing(mask):
        idx = np.flatnonzero(mask)[:list_max]
        sgn = np.sign(ref[idx])
        return [(int(i), float(ref[i]), float(got[i]), float(s * lo[i]), float(s * hi[i]), float(err[i]))
                for i, s in zip(idx, sgn)]

    return {"n": int(ref.size), "n_over": int(over.sum()), "n_format_limited": int(fmt.sum()),
            "n_rounding_side": int(side.sum()), "n_compute": int(comp.sum()),
            "max_abs": float(err.max()), "max_abs_rest": float(rest.max()),
            "max_before_rounding": float(before.max()),
            "rounding_side": listing(side), "format_limited": listing(fmt), "compute": listing(comp)}


def check_block_parity(name: str, got_bits: np.ndarray, ref: np.ndarray) -> dict:
    """The block-level bound (max-abs <= 2e-2 * RMS(ref), cosine >= 0.9995) on sampled outputs.

    Hard assertions: finite output; cosine; at most one element in 10^5 over the bound; and for
    every element the error minus half a bf16 spacing at the reference -- what the value must
    have carried before its final rounding -- within the bound.  The three classes of
    `tolerance_split` are printed and returned; the caller decides what to do when the raw
    bound itself is missed (see `expect_raw_bound`)."""
    st = stats(bits_to_f64(got_bits), ref)
    tol = 2e-2 * st["rms_ref"]
    sp = tolerance_split(got_bits, ref, tol)
    sp.update(name=name, rel=st["rel"], cos=st["cos"], rms_ref=st["rms_ref"], tol=tol,
              rel_rest=sp["max_abs_rest"] / st["rms_ref"], rel_before_rounding=sp["max_before_rounding"] / st["rms_ref"])
    print("%s: %d outputs, max-abs %.4e = %.4f of RMS (bound 0.02), cosine %.7f; over the bound %d: "
          "format-limited (exactly rounded reference fails) %d, rounding-side (faithful bf16, wrong side of a "
          "midpoint) %d, compute %d; max error before the final rounding >= %.4f of RMS"
          % (name, sp["n"], st["max_abs"], st["rel"], st["cos"], sp["n_over"], sp["n_format_limited"],
             sp["n_rounding_side"], sp["n_compute"], sp["rel_before_rounding"]))
    for kind in ("rounding_side", "format_limited", "compute"):
        for (i, r, g, lo, hi, e) in sp[kind]:
            print("    %s element %d: reference %.6f, gpu %.6f, bf16 neighbours %.6f / %.6f, error %.5f = %.4f of RMS"
                  % (kind, i, r, g, lo, hi, e, e / st["rms_ref"]))
    assert st["finite"], (name, "non-finite output")
    assert st["cos"] >= 0.9995, (name, st)
    assert sp["n_over"] <= max(1, 1e-5 * sp["n"]), (name, sp)
    assert sp["max_before_rounding"] <= tol, (name, sp)
    return sp


def expect_raw_bound(results) -> None:
    """Ends a test that has passed all its hard assertions: if any block-parity record misses
    the raw bound max-abs <= 2e-2 * RMS(ref), the test is reported as an expected failure with
    the measured figures (pytest.xfail), not as a pass."""
    import pytest
    if isinstance(results, dict):
        results = [results]
    missed = ["%s: raw max-abs %.4f of RMS; %d of %d outputs over the bound (%d rounding-side, %d format-limited, "
              "%d compute)" % (sp["name"], sp["rel"], sp["n_over"], sp["n"], sp["n_rounding_side"],
                               sp["n_format_limited"], sp["n_compute"])
              for sp in results if sp["rel"] > 2e-2]
    if missed:
        pytest.xfail("stated bound max-abs <= 2e-2 * RMS missed: " + "; ".join(missed))
