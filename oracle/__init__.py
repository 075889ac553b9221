"""CPU oracle of AMP training -- TEST INFRASTRUCTURE (tests, smoke check and the benchmark's CPU baseline only).

`Oracle` is a ctypes wrapper around ampnet_oracle.cpp; `build()` compiles it with g++.
"""
from .oracle import Oracle, build, OracleStats, round_bf16  # noqa: F401
