"""B200 (sm_100a) W4A8-dINT quantized linear layer: Python face of the C-ABI library.

The package is a thin binding (binding.py) over libw4a8.so plus the seeded synthetic
input generators (synth.py).  Importing it loads the CUDA library and fails if it has not
been built: there is no CPU or other fallback path.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    EXPORTS, LIB_PATH, PATH_AUTO, PATH_GEMV, PATH_SIMPLE, PATH_TCGEN05, Opts, W4A8Error, check_status,
    dint4_table, lib, linear, linear_acc_i32, linear_static, static_poll_status, linear_workspace_bytes, make_opts, new_workspace,
    pack_weights, packed_bytes, poll_status, quantize_act, unpack_codes, version,
    workspace_init, quantize_act_asym, weight_rowsum, linear_asym,
    quantize_linear, quantize_linear_workspace_bytes, new_quantize_linear_workspace, linear_plan,
    norm_quantize_act, NORM_RMS, NORM_LAYER, dint_table,
    pack_value, attn_pv, new_attn_pv_workspace,
    interleave_gate_up, linear_swiglu, new_linear_swiglu_workspace, linear_asym_group,
)
