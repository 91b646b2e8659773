"""Acceptance rule for floating-point outputs (oracle; tests only).

Every element of one rank's output must satisfy
``|gpu - ref| <= 1e-2 * max|ref| + 1e-3`` (BF16 output, FP32 accumulation),
with ``max|ref|`` taken over that rank's output tensor.  NaN or Inf on the
GPU side is a violation.  Because the bound is loose, the comparison also
reports the RMS error relative to the RMS of the reference and the fraction of
elements within one BF16 ulp of the correctly rounded reference; the tests
additionally require ``rms_rel <= 2**-8`` (times ``1 + 3 / sqrt(2 n)`` for a
tensor of n elements: three standard deviations of an RMS estimated from n
samples, which matters only below a few hundred elements).

A reduce-scatter ring whose messages are BF16 rounds its running sum once per
contributor; ``check_bf16_ring`` holds such a result against the hop-by-hop
reference (``operators.gemm_rs(..., bf16_hops=True)``) and, with limits that
account for the P roundings, against the exact sum.
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


def rms_limit(n: int, base: float = RMS_REL_LIMIT) -> float:
    return base * (1.0 + 3.0 / (2.0 * max(int(n), 1)) ** 0.5)


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
    return Report(ok=(violations == 0 and rms_rel <= rms_limit(ref.size)), violations=violations,
                  max_abs_err=max_err, tol=tol, max_ref=mref, rms_rel=rms_rel,
                  frac_within_1ulp=within, worst_index=tuple(int(i) for i in worst))


@dataclass
class RingReport:
    ok: bool
    identical: float            # fraction of elements equal to the hop-by-hop reference, bit for bit
    min_identical: float
    hops: Report                # against the hop-by-hop reference (tolerance from max|exact|)
    exact: Report               # against the exact sum
    allowed_beyond_bound: int

    def __str__(self) -> str:
        return (f"ok={self.ok} identical={self.identical:.5f} (>= {self.min_identical:.5f}) | vs hops: {self.hops} | "
                f"vs exact (<= {self.allowed_beyond_bound} beyond the bound): {self.exact}")


def check_bf16_ring(gpu_bits: np.ndarray, exact: np.ndarray, hops: np.ndarray, P: int, K: int,
                    max_ref: float | None = None) -> RingReport:
    """A GEMM+ReduceScatter result whose running sum was rounded to BF16 after every contributor.

    Against ``hops`` (the same ring computed hop by hop in the schedule's order, every hop's addition in FP32 and its
    rounding to BF16, partial products exact): the roundings are the same decisions on both sides except where the
    GPU's FP32 accumulation of a K-term partial falls on the other side of a rounding boundary than the exact partial.
    That happens to a fraction of about 1e-6 * K of the elements (a relative accumulation error of some K * 2^-24
    against rounding intervals of 2^-8); a different ORDER of the contributors changes a quarter of the elements.
    Required: at most max(1e-3, 3e-6 * K) of the elements not identical (as a count: the expected number plus three
    Poisson standard deviations, rounded up, so that a tensor of a few hundred elements may hold a flip), every element within the
    acceptance bound, RMS difference at most 2^-11 of the RMS of the result (2^-9 for tensors below 4096 elements,
    where one flipped rounding is a visible share of the whole).

    Against ``exact``: P roundings of up to 2^-8 relative each (RMS about 2^-9.3 each) cannot promise
    1e-2 * max|ref| on every element -- the worst case is P * 2^-8 -- and do not: at P = 8 about one element in
    1e7..1e8, among the largest of its tensor, lands a few per cent beyond the bound; at P = 16 (standard deviation
    of an element in the top binade about 0.4 of the bound) a few in 1e5 of a large tensor, up to 2 in 1e4 of a small one.
    Required: RMS error at most sqrt(P) * 2^-9 (2^-8 at least; times 1 + 3 / sqrt(2 n) for a tensor of n elements,
    three standard deviations of an RMS estimated from n samples, which matters below a few hundred elements), no
    error beyond twice the bound, and at most 1e-5 (P <= 8) or 1e-3 (P > 8) of the elements (counted like the
    flips above) beyond the bound."""
    mref = float(np.max(np.abs(exact))) if max_ref is None else float(max_ref)
    against_hops = check(gpu_bits, hops, max_ref=mref)
    against_exact = check(gpu_bits, exact, max_ref=mref)
    identical = float(np.mean(bf16_bits_to_f64(gpu_bits) == hops)) if hops.size else 1.0
    min_identical = 1.0 - max(1e-3, 3e-6 * K)
    def count_limit(rate, n):
        return int(np.ceil(rate * n + 3.0 * (rate * n) ** 0.5))
    allowed = count_limit(1e-5 if P <= 8 else 1e-3, exact.size)
    differing = int(np.sum(bf16_bits_to_f64(gpu_bits) != hops))
    few_differ = differing <= count_limit(1.0 - min_identical, hops.size)
    ok = (few_differ and against_hops.violations == 0 and against_hops.rms_rel <= 2.0 ** (-11 if hops.size >= 4096 else -9)
          and against_exact.rms_rel <= rms_limit(exact.size, max(RMS_REL_LIMIT, 2.0 ** -9 * P ** 0.5))
          and against_exact.max_abs_err <= 2.0 * against_exact.tol and against_exact.violations <= allowed)
    return RingReport(ok=ok, identical=identical, min_identical=min_identical, hops=against_hops,
                      exact=against_exact, allowed_beyond_bound=allowed)
