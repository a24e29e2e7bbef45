"""B200 (sm_100a) implementation of the LQER / L2QER inference linear layer.

The package is a thin ctypes binding over the C ABI declared in include/lqer.h;
every step of the layer runs in the CUDA library.  There is no CPU fallback:
loading fails loudly when the library has not been built.
"""
from .binding import (  # noqa: F401
    LqerError,
    Config,
    PackedWeights,
    lib,
    lib_path,
    default_config,
    packed_bytes,
    workspace_bytes,
    call_workspace_bytes,
    set_wait_limit_cycles,
    inject_stall,
    prepare_weights,
    prepare_from_calibration,
    factor_sketch_columns,
    export_weights,
    quantize_activations,
    project_lowrank,
    new_workspace,
    linear,
    linear_ex,
    linear_batched_ex,
    linear_batched,
    batched_workspace_bytes,
    linear_static,
    linear_host,
    linear_host_batched,
    linear_host_batched_ex,
    linear_host_batched_bytes,
    make_host_calls,
    poll_status,
    set_path,
    launch_count,
    profile_enable,
    profile_collect,
    make_calls,
)
