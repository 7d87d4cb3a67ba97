"""CPU oracle for the full-FP4 Direct-P attention forward.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 NumPy restatement of what the hot path
computes, written from the paper.  It shares no code with the CUDA path and must never
be imported by the product package; only tests, the smoke check and the benchmark's
cpu-baseline leg may call it.

Pinned by tests/test_oracle_*.py (run with -m "not gpu"):
  formats.py    E2M1 / E8M0 / E4M3 coders      -> printed codebook and boundaries, exhaustive
                                                  enumeration, closed forms, Table "p-range"
  quantize.py   MXFP4 / NVFP4 operand quantizers -> closed forms, brute force, error bounds; the three
                                                  amplitude rules -> exact rational arithmetic on every
                                                  bf16 significand, hand-computed blocks, saturation;
                                                  MSE rule -> block errors in exact rational arithmetic,
                                                  its fp32 summation order operation by operation;
                                                  per-(batch, head) NVFP4 factors -> power-of-two scaling
                                                  of a head moves only its factor, error bound per head
  attention.py  tiled Direct-P forward          -> tile-size / tile-order invariance, V == 1,
                                                  equal keys, dominant key, brute-force exact
                                                  attention on losslessly representable inputs;
                                                  affine code map -> its printed decision boundaries
                                                  (t_j - B)/A, the same invariants, the paper's
                                                  all-MXFP4 accuracy band; threshold amplitude rule
                                                  -> closed form, Table "p-range" MXFP4 row; causal mask
                                                  and grouped-query attention -> first row, whole-tile
                                                  prefixes, brute force, repeated K/V heads; mixed map
                                                  -> position by position against the two pinned maps,
                                                  error monotone in the share of exact pairs; per-head
                                                  factors -> bit-identical output under 2^a / 2^-a scaling
                                                  of a query head and its key head;
                                                  FP8 P/V route (E4M3 V per unit, E4M3 probabilities against the
                                                  integer row maximum) -> the E4M3 grid written out independently,
                                                  ties, saturation; closed forms of the V factor; representable
                                                  probabilities against brute force; constant V, flushing, key
                                                  permutation, causal prefix; the accuracy level the paper reports
"""
