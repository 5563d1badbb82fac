"""B200 (sm_100a) implementation of the constrained-MMSE quantization search of arXiv:1902.06822.

``binding`` wraps the C interface of include/omse.h (libomse.so, built by ``build``);
``synth`` generates the seeded synthetic tensors used by the tests and the benchmark.
"""
