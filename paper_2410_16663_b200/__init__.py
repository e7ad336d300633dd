"""B200 (sm_100a) fused attention forward: prefill and split-KV decode behind a C ABI.

``paper_2410_16663_b200.binding`` loads the CUDA shared library and exposes its entry
points under the same names; ``paper_2410_16663_b200.inputs`` holds the seeded synthetic
workloads.  Importing this package loads nothing; the binding raises if the library has not
been built (``python -m paper_2410_16663_b200.build``).
"""
__all__ = ["binding", "build", "inputs"]
