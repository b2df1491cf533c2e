"""CPU oracle for the online W4A4 WUSH linear layer (arXiv 2512.00956).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, fp64 restatement of
what the hot path computes, written from the paper.  It shares no code with the
CUDA library and must never be imported by it.  Only the test-suite, the smoke
check and the CPU-baseline leg of the benchmark may import it.

Pinned parts (each has CPU tests that compare it with something other than
itself): E2M1 / E8M0 / E4M3 / bf16 codecs (against ml_dtypes and brute force),
the Sylvester-Hadamard matrix (against scipy and H H^T = I), the transform
construction of Algorithm 1 (identities of Eq. 6, Appendix "equalization
effect", the diagonal closed form, Lemma A.1 and the Monte-Carlo optimum of
Theorem 4.1), the pre-quantisation invariance W x = (W T^-1)(T x), and the
dequantised product (exact rational arithmetic on tiny shapes), and the GPTQ case of
Algorithm 2 (gptq.py: the inter-block step in exact rationals, the intra-block subroutine
and the whole layer against the closed-form optimal compensation computed from the Hessian
by linear solves, the reduction to the RTN case for a block-diagonal Hessian).

Parity unpinned (conventions of this build; the paper is silent): the damping
ratio lambda = 0.01, the choice between the floor rule (default) and the ceil
rule ("mxfp4_ceil") of the MXFP4 shared exponent, the choice between the static
(calibration-time, default) and the per-batch NVFP4 activation tensor scale,
the fp32 operation order of the NVFP4 block scale, and, in the GPTQ case, when a
group's scale is fixed (at the block's turn, from its current values) and where the NVFP4
weight tensor scale comes from (an input).  (Each rule itself is pinned: only which one
the paper's authors used is not.)
"""
