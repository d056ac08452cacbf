"""CPU oracle for one Speculative Jacobi Decoding (SJD) iteration.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the SJD hot path computes (paper Sec. 3.1, Sec. 4.1 Steps 1-4, Eqs. 1-3,
Sec. 4.2, Appendix A).  It shares no code with the CUDA path and is imported
only by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
The product (the CUDA library and its Python binding) never imports it.

Modules
  philox    Philox4x32-10 counter-based generator (Salmon et al., SC'11).
  sampling  logit warp (temperature, top-k, softmax), inverse-CDF sampler,
            the verification scan of Eqs. 1-3.
  model     Llama-style decoder forward pass (the "auto-regressive
            transformer" of Sec. 3.1) with and without a KV cache.
  sjd       the SJD state machine (Steps 1-4), plus plain auto-regressive
            and greedy Jacobi decoding (Sec. 3.1, Sec. 3.2).

Pins (see tests/test_oracle_*.py): Philox known answers; W=1 equals ordinary
sampling; top-1 equals greedy Jacobi / greedy auto-regressive decoding;
forward passes never exceed tokens; chi-square exactness of single tokens and
of the joint distribution by brute-force enumeration; the identities of
Appendix A; window forward with cache equals the full causal forward; library
cross-checks of attention / normalisation / softmax.

Parity unpinned: acceptance *rates* and step compression on random-init
models cannot be pinned to the paper's Table 1/2 figures (those need trained
weights); only the algorithmic invariants above are pinned.
"""
