"""Swimba (Switch Mamba) token-mixer forward for NVIDIA B200 (sm_100a).

The hot path lives in the C-ABI library built from `csrc/` (see
`include/swimba.h`); `binding` is the thin ctypes layer over it and `synth`
draws the seeded synthetic inputs used by the tests and the benchmark.
"""
