"""CPU checker for the speculate-and-verify step.  TEST INFRASTRUCTURE, NOT PRODUCT.

Everything in this package is a plain, slow, obviously-correct restatement of what the step computes
(SuffixDecoding as the paper uses it: Section 3 overview and Section 3.3 "SuffixDecoding"): brute-force
occurrence scans instead of an index, direct tree construction from occurrence lists, fp64 attention,
acceptance by enumerating root paths.  It shares no code with the CUDA path and imports nothing from it.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it; the product never does.
"""
