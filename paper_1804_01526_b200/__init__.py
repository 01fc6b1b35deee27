"""HBFP dot-product path for B200: BFP quantisation and BFP GEMMs behind a C ABI.

``binding`` wraps ``libhbfp.so`` (built by ``paper_1804_01526_b200.build``); ``workloads`` holds
the seeded synthetic inputs and GEMM shapes of the benchmark configurations.
"""
from . import workloads  # noqa: F401

__all__ = ["binding", "build", "workloads"]
