"""B200-native OSDN layer: thin Python binding over the C ABI in ``include/osdn.h``.

The binding only marshals arguments (torch tensors -> device pointers); every step
of the layer runs in the CUDA kernels of ``libosdn.so``.  There is no CPU or eager
fallback: if the library is missing or no CUDA device is present the calls raise.

    from paper_2605_13473_b200 import osdn_fwd, osdn_bwd, osdn_precond_update
"""
from .binding import (  # noqa: F401
    OsdnParams,
    load_library,
    make_params,
    osdn_bwd,
    osdn_fwd,
    osdn_fwd_static,
    osdn_decode_step,
    osdn_precond_update,
    osdn_residual_ratio,
    osdn_step_host,
    osdn_workspace_bytes,
    osdn_host_staging_bytes,
    osdn_last_launch_count,
    osdn_read_device_status,
    status_string,
    run_inputs_fwd,
    run_inputs_bwd,
)
