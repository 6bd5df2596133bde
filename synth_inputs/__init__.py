"""Seeded synthetic inputs shared by the tests, the oracle runs and the benchmark.

This package only produces INPUTS (logit streams and constraint sets).  It holds none of the method's
arithmetic: no softmax, no selection, no constraint bookkeeping.  The logit generator exists twice, as
numpy code (``logits.py``) and as a CUDA kernel (``gen.cu``), built so that both write the same bits.
"""
from .configs import CONFIGS, Workload, make_workload  # noqa: F401
from .logits import LogitStream  # noqa: F401
