"""CPU oracle for the AWE exact integer matrix product.  TEST INFRASTRUCTURE ONLY.

Everything in this package is a plain, slow, CPU restatement of what the paper's
method computes: the storable set S and its E2M1 codes (Section 3.1), schemes and
admissible tuples (Definition 4.1), the run-time procedure (Algorithm 1), the
exact-accumulation bound K* (Section 3.4), the residue form (Section 5.3) and the
printed encodings (Appendix A).  It shares no code with the CUDA library and must
never be imported by the product path: only the tests, the smoke check and the
benchmark's CPU-baseline / reference arm may use it.

Parity pins live in tests/test_oracle_*.py.  One item is "parity unpinned":
the paper's totals of 59 (this method) and 75 (prior work) products for the FP64
significand cannot be recomputed because the list of three-product moduli they
rely on is not printed; see oracle/rns.py.
"""
