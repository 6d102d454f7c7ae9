"""CPU oracle for the speculative-decoding verify path (fp32, numpy).

TEST INFRASTRUCTURE ONLY.  Only tests, the smoke check and the benchmark's CPU-baseline /
reference legs may import this package; the product path never does, and this package
imports nothing from the CUDA path.
"""
