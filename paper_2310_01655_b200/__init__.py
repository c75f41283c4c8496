"""Causal polynomial-sketch (Polysketch) attention for B200: Python binding of libpsk.

The binding only marshals arguments (pointers, shapes, strides, stream) into the
C ABI declared in include/psk.h; every step of the computation runs in the library's
CUDA kernels.  There is no CPU or PyTorch fallback: if libpsk.so is missing or no CUDA
device is present the calls raise.
"""
from . import binding
from .binding import (PskError, Shape, lib, library_path, sketch, lt_multiply, lt_multiply_bf16, decode_state, decode_step, causal_attn_fwd, causal_attn_bwd, causal_attn_fwd_static,
                      static_scratch_bytes,
                      workspace_bytes, check, last_launch_count, status_string,
                      profile_enable, profile_records,
                      PATH_AUTO, PATH_CUDA_CORES, PATH_TENSOR_CORES, FLAG_KEEP_STATES,
                      FLAG_LOCAL_EXACT, FLAG_NONCAUSAL)

__all__ = ["PskError", "Shape", "lib", "library_path", "sketch", "lt_multiply", "lt_multiply_bf16", "decode_state", "decode_step", "causal_attn_fwd", "causal_attn_bwd", "causal_attn_fwd_static",
           "static_scratch_bytes",
           "workspace_bytes", "check", "last_launch_count", "status_string",
           "profile_enable", "profile_records",
           "PATH_AUTO", "PATH_CUDA_CORES", "PATH_TENSOR_CORES", "FLAG_KEEP_STATES",
           "FLAG_LOCAL_EXACT", "FLAG_NONCAUSAL"]
