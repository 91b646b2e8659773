"""CPU oracle for the fused AllGather+GEMM / GEMM+ReduceScatter hot path.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, obviously-correct
restatement of what the paper's operators compute (numpy, FP64).  It shares no
code with the CUDA library and is never imported by it.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may use it.

Modules
-------
schedule   double/single ring chunk order, closed form (Section III-A/III-B)
ring_sim   the same tables obtained by simulating token passing on the rings
operators  AllGather+GEMM, GEMM+ReduceScatter, InterDecom(d) in FP64
models     Eq. 2-5 (decomposition model, optimal degree), Eq. 7-8 (fusion
           model), Algorithm 1 (strategy selector), calibration regressions
compare    the acceptance rule |gpu - ref| <= 1e-2 * max|ref| + 1e-3
mlp        the tensor-parallel MLP block of Section II-A (both collectives through
           ``operators``, activation in FP64, one rounding of the intermediate)

Pins (what each part is checked against, other than itself) live in
``tests/test_oracle_*.py``.  Parts whose *numerical agreement with the paper's
own predictions* cannot be pinned because the paper prints no calibrated
parameters: ``models.decomp_time`` / ``models.fusion_time`` / ``models.select``
are pinned by algebraic special cases and hand-evaluated examples only
("parity unpinned" against the paper's Table II and MAE figures).
"""

OP_AG_GEMM = 0
OP_GEMM_RS = 1
