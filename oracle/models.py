"""Performance models and the strategy selector (oracle; tests only).

Follows Section IV (Eq. 2-5), Section V-B (Eq. 7-8) and Algorithm 1, step by
step and in the paper's notation.  Numerical agreement with the paper's own
predictions is *parity unpinned*: the paper prints no calibrated
alpha/beta values.  These functions are pinned by the algebraic facts the
paper states (T(1) = T_comp + T_comm; eta = 1 gives the overhead-agnostic
model; convexity, so the analytic optimum equals the enumerated one) and by
hand-evaluated examples.

Readings where the text is silent or prints one regime only:

* Eq. 5 is printed with 1/lambda, which is the derivative condition of Eq. 2
  when T_comp >= T_comm.  Setting dT/dd = 0 in general gives
  d^2 = ((T_comp + T_comm)/max(T_comp, T_comm) - alpha)/beta, i.e. the printed
  formula with rho = min(lambda, 1/lambda) in place of 1/lambda.  ``rho`` is
  used by default; ``as_printed=True`` evaluates the formula literally.
* P_2 rounds to the nearest power of two on a log scale (exact ties go to the
  smaller power), which is where a convex A*d + B + C/d changes its better
  neighbour; the result is clamped to the paper's candidate set {2,4,8,16}
  and to ``d_max`` (the largest degree the rows divide by).
* A non-positive beta or radicand has no analytic candidate: the candidate is
  then the argmin of Eq. 2 over the candidate set.  T_comm <= 0 gives d = 1.
* Eq. 7: equal chunks, T_comp^chunk = T_comp / n; the collective moves data
  during n-1 steps, T_comm^chunk = T_comm / (n-1); n_chunks = number of GPUs.
* Ties: Eq. 4 and Algorithm 1 use strict "<"; equal times keep d = 1 and
  select InterDecom respectively.
* T_comp and T_comm are linear in the work: T_comp = a + b*FLOPs,
  T_comm = a' + b'*bytes, FLOPs = 2*P*M*N*K over all ranks and
  bytes = 2*P*M*K (AllGather) or 2*P*M*N (ReduceScatter).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Optional, Sequence, Tuple

from . import OP_AG_GEMM, OP_GEMM_RS

CANDIDATE_DEGREES = (2, 4, 8, 16)          # Table IV, "Decomposition Degree"
STRATEGY_INTRAFUSION = 0
STRATEGY_INTERDECOM = 1


@dataclass(frozen=True)
class Calib:
    comp_a: float = 0.0       # T_comp = comp_a + comp_b * FLOPs
    comp_b: float = 0.0
    comm_a: float = 0.0       # T_comm = comm_a + comm_b * bytes
    comm_b: float = 0.0
    alpha_decomp: float = 1.0
    beta_decomp: float = 0.0
    alpha_fusion: float = 0.0
    beta_fusion: float = 0.0


def eta_decomp(d: int, alpha: float, beta: float) -> float:
    """Eq. 3."""
    return alpha + beta * d


def decomp_time(t_comp: float, t_comm: float, alpha: float, beta: float, d: int) -> float:
    """Eq. 2 with T_stage = max(T_comp/d, T_comm/d) and the non-overlapped
    portion T_comp/d + T_comm/d."""
    t_stage = max(t_comp / d, t_comm / d)
    overlapped = (d - 1) * t_stage * eta_decomp(d, alpha, beta)
    return overlapped + t_comp / d + t_comm / d


def nearest_power_of_two(x: float) -> int:
    """P_2: nearest power of two on a log scale, ties to the smaller."""
    if not (x > 0.0) or math.isinf(x):
        raise ValueError("P_2 needs a positive finite argument")
    lo = math.floor(math.log2(x))
    # guard against log2 rounding at exact powers of two
    while 2.0 ** lo > x:
        lo -= 1
    while 2.0 ** (lo + 1) <= x:
        lo += 1
    low, high = 2.0 ** lo, 2.0 ** (lo + 1)
    # log-nearest: x/low <= high/x  <=>  x*x <= low*high
    p = low if x * x <= low * high else high
    return int(p) if p >= 1 else 1


def d_continuous(t_comp: float, t_comm: float, alpha: float, beta: float,
                 as_printed: bool = False) -> Optional[float]:
    """The argument of P_2 in Eq. 5, or None when it does not exist."""
    if t_comp <= 0 or t_comm <= 0 or beta <= 0:
        return None
    lam = t_comp / t_comm
    rho = 1.0 / lam if as_printed else min(lam, 1.0 / lam)
    radicand = (1.0 - alpha + rho) / beta
    if radicand <= 0:
        return None
    return math.sqrt(radicand)


def feasible_degrees(d_max: int) -> Tuple[int, ...]:
    return tuple(d for d in CANDIDATE_DEGREES if d <= d_max)


def d_candidate(t_comp: float, t_comm: float, alpha: float, beta: float,
                d_max: int = 16, as_printed: bool = False) -> Optional[int]:
    """Eq. 5, clamped to the feasible candidate set; None if that set is empty."""
    cands = feasible_degrees(d_max)
    if not cands:
        return None
    x = d_continuous(t_comp, t_comm, alpha, beta, as_printed)
    if x is None:
        best = cands[0]
        for d in cands[1:]:
            if decomp_time(t_comp, t_comm, alpha, beta, d) < decomp_time(t_comp, t_comm, alpha, beta, best):
                best = d
        return best
    if x >= 2.0 * cands[-1]:                 # also covers an overflowed (infinite) argument
        return cands[-1]
    d = nearest_power_of_two(x)
    return min(max(d, cands[0]), cands[-1])


def optimal_degree(t_comp: float, t_comm: float, alpha: float, beta: float,
                   d_max: int = 16, as_printed: bool = False) -> int:
    """Eq. 4: keep the candidate only if it beats sequential execution."""
    if t_comm <= 0:
        return 1
    cand = d_candidate(t_comp, t_comm, alpha, beta, d_max, as_printed)
    if cand is None:
        return 1
    if decomp_time(t_comp, t_comm, alpha, beta, cand) < decomp_time(t_comp, t_comm, alpha, beta, 1):
        return cand
    return 1


def fusion_overhead(n_chunks: int, alpha_f: float, beta_f: float, m_volume: float) -> float:
    """Eq. 8."""
    return (n_chunks - 1) * (alpha_f + beta_f * m_volume)


def fusion_time(t_comp: float, t_comm: float, n_chunks: int,
                alpha_f: float, beta_f: float, m_volume: float) -> float:
    """Eq. 7."""
    t_comp_chunk = t_comp / n_chunks
    t_comm_chunk = t_comm / (n_chunks - 1) if n_chunks > 1 else 0.0
    total = 0.0
    for _i in range(2, n_chunks + 1):
        total += max(t_comp_chunk, t_comm_chunk)
    return total + t_comp_chunk + fusion_overhead(n_chunks, alpha_f, beta_f, m_volume)


def workload_flops(P: int, M: int, N: int, K: int) -> float:
    return 2.0 * P * M * N * K


def workload_comm_bytes(op: int, P: int, M: int, N: int, K: int) -> float:
    return 2.0 * P * M * (K if op == OP_AG_GEMM else N)


def message_volume(op: int, M: int, N: int, K: int) -> float:
    """m of Eq. 8: M*K for AllGather, M*N for ReduceScatter."""
    return float(M) * (K if op == OP_AG_GEMM else N)


def max_degree(M: int, P: int) -> int:
    rows = M // P
    d = 1
    while d < 16 and rows % (2 * d) == 0:
        d *= 2
    return d


@dataclass(frozen=True)
class Choice:
    strategy: int
    d_star: int
    t_fusion: float
    t_decomp: float
    t_comp: float
    t_comm: float
    lam: float
    t_star: float


def select(op: int, P: int, M: int, N: int, K: int, calib: Calib, as_printed: bool = False) -> Choice:
    """Algorithm 1.  ``as_printed`` evaluates Eq. 5 literally (1/lambda) inside it."""
    # Phase 1: base metrics
    t_comp = calib.comp_a + calib.comp_b * workload_flops(P, M, N, K)
    t_comm = calib.comm_a + calib.comm_b * workload_comm_bytes(op, P, M, N, K)
    lam = t_comp / t_comm if t_comm > 0 else math.inf
    # Phase 2: parameters and degree
    d_star = optimal_degree(t_comp, t_comm, calib.alpha_decomp, calib.beta_decomp, max_degree(M, P), as_printed)
    # Phase 3: prediction and selection
    t_decomp = decomp_time(t_comp, t_comm, calib.alpha_decomp, calib.beta_decomp, d_star)
    t_fusion = fusion_time(t_comp, t_comm, P, calib.alpha_fusion, calib.beta_fusion,
                           message_volume(op, M, N, K))
    if t_fusion < t_decomp:
        return Choice(STRATEGY_INTRAFUSION, d_star, t_fusion, t_decomp, t_comp, t_comm, lam, t_fusion)
    return Choice(STRATEGY_INTERDECOM, d_star, t_fusion, t_decomp, t_comp, t_comm, lam, t_decomp)


# ---- offline calibration (one-time linear regressions) ---------------------

def ols(xs: Sequence[float], ys: Sequence[float]) -> Tuple[float, float]:
    """Least-squares line y = a + b*x.  One distinct x gives (mean(y), 0)."""
    n = len(xs)
    if n == 0 or n != len(ys):
        raise ValueError("need matching, non-empty samples")
    mx = sum(xs) / n
    my = sum(ys) / n
    sxx = sum((x - mx) ** 2 for x in xs)
    if sxx == 0:
        return my, 0.0
    b = sum((x - mx) * (y - my) for x, y in zip(xs, ys)) / sxx
    return my - b * mx, b


def eta_measured(t_meas: float, t_comp: float, t_comm: float, d: int) -> float:
    """Invert Eq. 2 for the overhead factor at one measured point (d > 1)."""
    t_stage = max(t_comp, t_comm) / d
    return (t_meas - (t_comp + t_comm) / d) / ((d - 1) * t_stage)


def fit_decomp_overhead(samples: Sequence[Tuple[float, float, int, float]]) -> Tuple[float, float]:
    """samples: (T_comp, T_comm, d, T_measured) with d > 1 -> (alpha, beta)."""
    ds = [float(d) for (_c, _m, d, _t) in samples]
    etas = [eta_measured(t, c, m, d) for (c, m, d, t) in samples]
    return ols(ds, etas)


def fit_fusion_overhead(samples: Sequence[Tuple[float, float, int, float, float]]) -> Tuple[float, float]:
    """samples: (T_comp, T_comm, n_chunks, m_volume, T_measured) -> (alpha_f, beta_f):
    regress the per-synchronisation-point residual of Eq. 7 on m."""
    xs, ys = [], []
    for (c, m, n, vol, t) in samples:
        if n < 2:
            continue
        base = fusion_time(c, m, n, 0.0, 0.0, vol)
        xs.append(vol)
        ys.append((t - base) / (n - 1))
    return ols(xs, ys)
