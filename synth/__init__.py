"""Seeded synthetic workloads shaped like LLaVA decoding.

Input generation only: this package contains none of the method's arithmetic
(no attention, no scoring, no selection, no schedule evaluation).  Both the
CPU oracle's tests and the CUDA path's tests/benchmark draw their inputs here
so that they see bit-identical tensors.
"""
from .configs import WORKLOADS, Workload, get_workload  # noqa: F401
from .inputs import SynthInputs  # noqa: F401
