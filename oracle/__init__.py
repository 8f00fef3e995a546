"""Slow, plain fp64 CPU oracle for the CERAR coding pipeline.

THIS PACKAGE IS TEST INFRASTRUCTURE.  It exists so that the CUDA library can be
checked against something written directly from the paper.  It shares no code,
tables or helpers with the CUDA path, imports nothing from it, and nothing in
the product may import it: only the test-suite, the smoke check and the
benchmark's CPU-baseline leg call into it.

Contents
--------
protocol : chunking, encoding, the ring rounds from the update equations (and,
           as a cross-check, on the storage slots of Algorithm 1), the
           observation matrix Y_i, decoding, the matrices M_i(U), the
           least-squares objective Phi and the rate counters.
designs  : the coefficient constructions (multiplicative perturbation
           construction, Vandermonde, epsilon-construction, the
           condition-number-constrained alternating least squares heuristic).
mixed    : the ring rounds with bfloat16 or 8-bit (e4m3, power-of-two scale per
           tile of positions) messages: binary32 worker arithmetic, every
           transmitted vector rounded to nearest-even by its sender.

Pins (what each function is checked against, see tests/test_oracle_*.py):
  rounds / whole pipeline : brute-force composition Y_i = G^(i) M_i(U) for
      arbitrary U; the worked example N=4, c=5 (Fig. 1 and Sec. II-A).
  MPC / Vandermonde / epsilon designs : Prop. 1, Prop. 2, Theorem 1's closed
      form, Eq. (error_scaling), Theorem 2 / Corollary 1 scaling laws, the
      finite-difference identity (Lemma 2) and the printed F_3.
  kappa-constrained design : every step against its defining property (U- and
      R-step are stationary minimisers of the brute-force Phi, the projection is
      the nearest matrix with singular values in the interval), the order of the
      steps in the loop, the reported history, the fixed-point property of what is
      returned, and the known optimum Phi = 0 at c = N.  Which local solution is
      reached at c > N has no published counterpart: PARITY UNPINNED for that
      end point.
  8-bit messages : the e4m3 rounding against hand-worked values (ties, subnormals,
      clamping) and torch's float8_e4m3fn conversion bit for bit; the tile scales
      against their defining inequality; the rounds as for bfloat16.
  bfloat16 messages : the rounding against worked values, IEEE properties and
      torch's conversion; the rounds against Algorithm 1 where nothing rounds and
      against the error the message precision implies.
"""
