"""CPU oracle for the DScale verify-side hot path.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain statement of what
the three library calls compute, written from the paper (Algorithm 1,
Eq. 6-11, Eq. 15, the "Prefix verifier" paragraph, Algorithm 2).  It shares
no code with the CUDA library and must never be imported by the product
package; only the tests, the smoke check and the benchmark's CPU-baseline
leg may call it.

Modules
-------
dvl_alloc    literal Algorithm 1: prefix scores, seed, serial budget loop,
             offsets, flat-pack, sentinels.
verify_attn  the plain definition of packed verify attention (explicit
             masks, dense softmax), plus the unpacked W=16 formulation.
accept       first-index row argmax and the sequential acceptance loop.

Every function is pinned by tests that do not go through the function itself
(worked examples printed in the paper, closed forms, brute force, library
special cases); there is no "parity unpinned" function in this package.
"""
