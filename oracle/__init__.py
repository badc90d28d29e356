"""CPU oracle of the local update step (Sec. 3, Sec. 6 of the paper).

TEST INFRASTRUCTURE ONLY.  A plain, slow NumPy implementation used to check the CUDA path and to
give the benchmark its CPU baseline.  It shares no code with the CUDA path; the product never
imports it.  Pinned by tests/test_oracle_*.py against finite differences, an independent
reverse-mode differentiation (K=1 is back-propagation), closed forms and brute force.

Parity unpinned against the paper (it prints no value for them): the constants and readings listed
in oracle/local_step.py's header (eps, GELU form, initialisation, loss reduction, ramp-up policy).
"""
