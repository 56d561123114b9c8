"""CPU fp64 oracle for the TS-DP speculative denoising round (arXiv 2512.15773).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain definition of what the
CUDA path must compute.  It may be imported by the test-suite, by the smoke check
and by the benchmark's CPU-baseline leg -- never by the product package, which has
no CPU fallback and fails loudly when its CUDA library is missing.  It shares no
code with the CUDA path: the counter-based random generator, the DDPM tables and
both networks are written a second time here, in numpy fp64, from the paper's
equations (Sec. 3.1 Eqs. 1-3 and the reflection-coupling equations, Sec. 3.2
Eq. (3) and the log-acceptance-ratio equation) and from the textbook DDPM
posterior the paper refers to as "the DDPM scheduler".

Pin status (what checks each part against something other than itself):
  philox.py   pinned  : published known-answer vectors of Philox4x32-10.
  ddpm.py     pinned  : direct products, closed forms, the affine-Gaussian recursion.
  spec.py     pinned  : Gaussian log-density identity, Householder invariants,
                        closed-form acceptance rate 2*Phi(-|d|/2), brute-force
                        first-rejection enumeration, drafter==base == vanilla,
                        KS test against the analytic marginal of the sampler.
  nets.py     parity unpinned against the paper (its trained networks and exact
              layer layout are not published); the wiring of the library's own
              architecture definition IS pinned: attention against a library routine
              (scale, head partition, causal mask), a decoder block, an adaptive-LayerNorm
              block and a 2-level conv UNet element by element in plain loops, the
              modulation slices and FiLM halves through closed forms, plus structural
              invariants (causality, zero-weight behaviour) -- tests/test_oracle_nets*.py.
  sched.py    parity unpinned against the paper (Sec. 3.3 names the three input streams, the
              separate encoders, the aggregating MLP and the five outputs, but no sizes, weights
              or ranges); pinned by structure: zero network, output ranges, stream separation,
              a hand-computed path, the stage boundaries.
              The intermediate reward of Sec. 3.3 (process_reward) is pinned by worked values and by
              the accumulated-reward identity the paper states for its scaling factor.
  distill.py  pinned  : zero for equal networks, the closed form for a constant output offset
                        (with the printed values c_50 = 0.2145, c_1 = 1.735 of the linear schedule),
                        linearity in (lambda1, lambda2), the Gaussian-overlap integral.
                        Gradient step on the Gaussian drafter: central finite differences of that
                        loss (each term alone and the sum), zero gradient at the base's parameters,
                        monotone descent to them.
  spec.FrozenTargetDraft  parity unpinned against the prior work that Sec. 2.2 cites (only named
              there); pinned by: first draft exact, K = 1 == vanilla, the Gaussian chain's marginal.
  sigma_scale parity unpinned against the paper (formula not given there).
"""
