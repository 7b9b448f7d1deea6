"""CPU oracle for FP8 Delta-Matching attention.

TEST INFRASTRUCTURE ONLY.  Plain, slow numpy code in float64 that states what
the attention path computes, step by step, so that it can be checked against
the paper by eye.  It shares nothing with the CUDA path: no kernels, headers,
tables or helpers, and it never imports the product package.  Only the tests,
the smoke check and the benchmark's CPU-baseline leg may import it.

Modules
-------
mxfp8      block-scaling quantiser: E4M3 codes with one E8M0 scale per 32
           consecutive elements along a contraction dimension.
attention  reference attention (nothing quantised), the emulated-FP8 forward
           and backward with the Delta-Matching / stale-delta row correction,
           and the BF16-operand variant of the same path.

Pins (tests marked "not gpu"): scaled_dot_product_attention + autograd in
float64, central finite differences, the softmax Jacobian, closed forms,
torch's float8_e4m3fn / float8_e8m0fnu casts, brute-force nearest-value
search, and the row-sum / column-sum identities of the paper (Eq. 1, Eq. 2,
Eq. 4-5).  The exact values of O, dQ, dK, dV on the emulated-FP8 path have no
printed example in the paper: parity unpinned beyond construction (operands
replaced by their grid values in the pinned reference formulas) and a second,
loop-based restatement on tiny shapes.
"""
