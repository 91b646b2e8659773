"""Acceptance rule for floating-point outputs (oracle; tests only).

Every element of one rank's output must satisfy
``|gpu - ref| <= 1e-2 * max|ref| + 1e-3`` (BF16 output, FP32 accumulation),
with ``max|ref|`` taken over that rank's output tensor.  NaN or Inf on the
GPU side is a violation.  Because the bound is loose, the comparison also
reports the RMS error relative to the RMS of the reference and the fraction of
elements within one BF16 ulp of the correctly rounded reference; the tests
additionally require ``rms_rel <= 2**-8``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from .operators import bf16_bits_to_f64, f64_to_bf16_f64

RTOL_OF_MAX = 1e-2
ATOL = 1e-3
RMS_REL_LIMIT = 2.0 ** -8


@dataclass
class Report:
    ok: bool
    violations: int
    max_abs_err: float
    tol: float
    max_ref: float
    rms_rel: float
    frac_within_1ulp: float
    worst_index: tuple

    def __str__(self) -> str:
        return (f"ok={self.ok} violations={self.violations} max_abs_err={self.max_abs_err:.4g} "
                f"tol={self.tol:.4g} max_ref={self.max_ref:.4g} rms_rel={self.rms_rel:.3g} "
                f"within_1ulp={self.frac_within_1ulp:.4f} worst={self.worst_index}")


def check(gpu_bits: np.ndarray, ref: np.ndarray, max_ref: float | None = None) -> Report:
    """gpu_bits: uint16 BF16 patterns; ref: FP64, same shape.  ``max_ref``
    overrides max|ref| when ``ref`` is only a sample of the rank's tensor."""
    assert gpu_bits.shape == ref.shape, (gpu_bits.shape, ref.shape)
    got = bf16_bits_to_f64(gpu_bits)
    mref = float(np.max(np.abs(ref))) if max_ref is None else float(max_ref)
    tol = RTOL_OF_MAX * mref + ATOL
    finite = np.isfinite(got)
    err = np.where(finite, np.abs(got - ref), np.inf)
    bad = ~(err <= tol)
    violations = int(bad.sum())
    worst = np.unravel_index(int(np.argmax(err)), err.shape) if err.size else ()
    ferr = np.where(finite, got - ref, 0.0)
    rms_ref = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    rms_err = float(np.sqrt(np.mean(ferr * ferr))) if ref.size else 0.0
    rms_rel = rms_err / rms_ref if rms_ref > 0 else (0.0 if rms_err == 0 else np.inf)
    rounded = f64_to_bf16_f64(ref)
    ulp = np.maximum(np.abs(rounded), 2.0 ** -126) * 2.0 ** -7      # >= one BF16 ulp at that magnitude
    within = float(np.mean(np.abs(np.where(finite, got, np.inf) - rounded) <= ulp)) if ref.size else 1.0
    max_err = float(np.max(err)) if err.size else 0.0
    return Report(ok=(violations == 0 and rms_rel <= RMS_REL_LIMIT), violations=violations,
                  max_abs_err=max_err, tol=tol, max_ref=mref, rms_rel=rms_rel,
                  frac_within_1ulp=within, worst_index=tuple(int(i) for i in worst))
