"""CPU oracle for routed structured-sparse causal prefill attention (RouteSparse).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain restatement of what the CUDA
path computes, written from the paper's definitions in float64 numpy.  It is imported only
by the tests, by the smoke check and by the benchmark's CPU-baseline leg; the product
path never calls it, and it imports nothing from the CUDA package.

Parts and what pins them (tests/test_oracle_*.py):
  attention.dense_attention      Eq. 1, plain definition.        Pinned: row 0, K=0 mean, torch SDPA.
  attention.masked_attention     Section 2.1 masked variant.      Pinned: causal mask == dense, LSE merge, explicit bitset.
  probe.probe                    Eq. 3 in the last-64-query form. Pinned: row sums, brute force vs the full matrix A.
  patterns.*                     Section 3.1 pattern library.     Pinned: brute-force pair counts, coverage vs plain
                                                                  definition, nesting, k >= n.  The concrete tie-break
                                                                  and the block expansion of slashes are this build's
                                                                  reading: beyond those invariants "parity unpinned".
  routing.route                  Eq. 4, Eq. 6-8, fallback.        Pinned: constraints, trivial budgets, exhaustive optimum
                                                                  as a lower bound.  The exact substitution order is this
                                                                  build's reading: "parity unpinned".
  certificate.certificate        Eq. 5.                           Pinned: equality case, L1 identity, bound on every row.
  probe.pooled_probe             Eq. 3, general form + descriptors. Pinned: width 1 == exact probe, per-key brute force,
                                                                  identical keys -> uniform rows, agreement and signature
                                                                  bins in a closed-form case (sink rows against uniform
                                                                  rows).  The proportions of the mixture and the pooling of
                                                                  a straddling block are this build's reading.
  probe.probe_rows(starts=...)   Eq. 3 at key resolution on four 16-row runs of the query mixture.  Pinned: brute force
                                                                  against the full attention matrix; the last-64-row runs
                                                                  give the ordinary probe bit for bit.
  patterns.mixture_coverage_fx   coverage on the mixture's rows.   Pinned: closed cases (whole blocks, half blocks, columns).
                                                                  The even split of a block's mass over its visible keys
                                                                  is this build's reading: "parity unpinned".
  calibration.*                  Section 3.5, predictor e of Eq. 4. Pinned: isotonic fit == scikit-learn's, quantile by
                                                                  counting, monotonicity.  The feature set is this build's
                                                                  reading: "parity unpinned".
  projection.qkv_project         the producer of Q, K, V (Section 3.4: routing beside the projection kernels).
                                                                  Pinned: torch linear + rotate-half, rotation special cases,
                                                                  distance-only dot products, brute-force side outputs.
"""
from . import attention, calibration, certificate, patterns, probe, projection, routing  # noqa: F401
