"""LinSimp (linearized 2-simplicial attention) hot path for B200: thin binding over liblinsimp.so.

Every step of the path runs in the library's CUDA kernels; this package only
marshals arguments.  There is no CPU or PyTorch fallback: calling an op without
the built library or without a CUDA device raises.
"""
from .binding import (LinSimpError, Params, decode_step, fwd, bwd, last_launch_count, lib_path,
                      load_library, workspace_bytes, BF16, F32, ALGO_DEFAULT, ALGO_FP32,
                      OP_FWD, OP_BWD, OP_DECODE, OP_STATE, prefill_state, decode_prepare, fwd_continue, bwd_continue, fwd_packed, bwd_packed, ring_fill_packed, winsimp_fwd, ring_fill, profile_enable,
                      profile_read, OP_NORM, qkr_normalize, qkr_normalize_bwd, gate_rmsnorm, gate_rmsnorm_bwd,
                      fwd_padded, bwd_padded, ring_fill_padded)
from .head import LinSimpHead, head_fwd, head_bwd

__all__ = ["LinSimpError", "Params", "decode_step", "fwd", "bwd", "last_launch_count", "lib_path",
           "load_library", "workspace_bytes", "BF16", "F32", "ALGO_DEFAULT", "ALGO_FP32",
           "OP_FWD", "OP_BWD", "OP_DECODE", "OP_STATE", "prefill_state", "decode_prepare", "fwd_continue", "bwd_continue", "fwd_packed", "bwd_packed", "ring_fill_packed", "winsimp_fwd", "ring_fill", "profile_enable",
           "profile_read", "OP_NORM", "qkr_normalize", "qkr_normalize_bwd", "gate_rmsnorm", "gate_rmsnorm_bwd", "fwd_padded", "bwd_padded", "ring_fill_padded",
           "LinSimpHead", "head_fwd", "head_bwd"]
