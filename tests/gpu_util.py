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


def tolerance_split(got_bits: np.ndarray, ref: np.ndarray, tol: float):
    """Classifies the elements whose error exceeds `tol`.

    A bf16 result is *faithfully rounded* when it is one of the two bf16 numbers that bracket
    the reference.  Where the bf16 spacing is larger than the tolerance (|y| >= 4 for
    tol = 2e-2 * RMS with RMS ~ 1.1), a faithfully rounded result can still be off by up to
    one spacing: passing would need the pre-rounding value to fall on the correct side of a
    rounding midpoint, which no bf16-input arithmetic can promise.  Those elements are
    format-limited; every other element over the tolerance is a compute violation.
    Returns (n_over, n_format_limited, n_compute, max_abs_compute_only)."""
    got = bits_to_f64(got_bits).ravel()
    ref = np.asarray(ref, np.float64).ravel()
    err = np.abs(got - ref)
    over = err > tol
    r32 = ref.astype(np.float32)
    mag = r32.view(np.uint32) & np.uint32(0x7FFFFFFF)
    lo = (mag & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    hi = ((mag & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    exact = (mag & np.uint32(0xFFFF)) == 0
    g = np.abs(got)
    same_sign = (np.signbit(got) == np.signbit(ref)) | (got == 0)
    faithful = same_sign & ((g == lo) | ((g == hi) & ~exact))
    fmt = over & faithful
    comp = over & ~faithful
    masked = np.where(fmt, 0.0, err)
    return int(over.sum()), int(fmt.sum()), int(comp.sum()), float(masked.max())
