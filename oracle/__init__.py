"""CPU oracle for the HLQ bit-serial LUT GEMM/GEMV (test infrastructure).

This package is TEST INFRASTRUCTURE, not part of the product: only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import it.
It is a plain, slow, fp64 restatement of what the path computes, written from
the paper's definitions, and it shares no code with the CUDA library.

Modules
-------
hlq      the definition: W_hat = sum_j s_j b_j + z (Eq. 3 / Eq. 6, per-group
         parameters as in Algorithm 1) and Y = X W_hat^T, the offset-only term,
         and the bit-plane split of the worked example (Appendix B)
lut      the same result through the bit-serial look-up-table procedure of
         Appendix B (tables of 2^g partial sums, look-up, per-group scale),
         and the mirror (+-1) form of Appendix D
storage  bits-per-weight and model-size accounting (Tables 1 and 3 of the paper)
fit      Algorithm 1 (alternating bit-pattern selection and least squares) that produces
         (B, s, z) from unquantised fp16 weights
layout   reference packer / unpacker for the library's device layout
         (a documented pure function; the paper fixes no device layout, so
         this part is "parity unpinned" by the paper and pinned by round trip,
         bijectivity and a consumer walk against the definition)

Pins: every function here is checked by `tests/test_oracle_*.py` against
something other than itself (the paper's worked example and printed sizes,
exact rational brute force, the uniform closed form, library matmul).
"""
