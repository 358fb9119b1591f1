"""CPU oracle (test infrastructure): plain definitions the CUDA path must match bit for bit.

`oracle.gcm` wraps the C file gcm_oracle.c (AES-128, CTR, GHASH, GCM, segment semantics);
`oracle.labels` is the ownership-label join and the four flow rules in plain Python.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package;
it never imports the CUDA binding.
"""
