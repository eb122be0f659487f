"""B200-native batched multi-draft greedy block verification (SpecTr-GBV verify step).

The work is done by hand-written sm_100a CUDA kernels behind a C-ABI shared library
(``csrc/libsgbv.so``, declared in ``include/sgbv.h``); :mod:`.binding` marshals torch tensors
into that ABI.  There is no CPU fallback: calling a verify function without the built library
or without a CUDA device raises.
"""
from .workloads import CONFIGS, VerifyConfig, VerifyInputs, get_config, make_inputs, make_uniforms, sweep_c5  # noqa: F401

__all__ = ["CONFIGS", "VerifyConfig", "VerifyInputs", "get_config", "make_inputs", "make_uniforms",
           "sweep_c5"]
