"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This package holds *inputs only*: the integer codes of the IR description
format, the four canonical IR graphs as plain node/edge tables, the seeded
instance generators and the seeded parameter initialisers.  It contains none
of the training method's arithmetic (no forward/backward of the trained
model, no update rule, no scheduling); both implementations consume what it
produces and neither is imported by it.
"""
from . import ir, data, params  # noqa: F401
