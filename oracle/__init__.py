"""CPU oracle for the UniPool MoE-layer hot path.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
directory; the only callers are the test-suite, the smoke check and the
benchmark's CPU-baseline leg.  The oracle shares no code with the CUDA path
and imports nothing from it: it depends on numpy and the standard library.

Modules
-------
unipool_oracle   vectorised numpy statement of the paper's equations
                 (Eq. 2 layer, Eq. 7 NormRouter, Eqs. 3-6 balance losses) and
                 of their derivatives.
brute            the same forward pass as explicit per-token Python loops over
                 plain floats; used to pin ``unipool_oracle`` on tiny inputs.
norm_router_c    Monte-Carlo estimate of the NormRouter constant c (Alg. 1).
"""
