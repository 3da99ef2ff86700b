"""B200 (sm_100a) library for the fully quantized forward pass of a sinusoidal INR (DHQ).

The work is done by hand-written CUDA kernels behind the C ABI of `include/dhq.h`; this package
is the thin Python binding over that shared library.  There is no CPU or PyTorch fallback: if the
library has not been built (`python -m paper_2508_13478_b200.build`), importing the binding's
functions raises.
"""
from .binding import (  # noqa: F401
    DHQ_GRAN_TENSOR, DHQ_GRAN_CHANNEL_OR_TOKEN, DHQ_ROT_INPUT, DhqError, PIPES,
    dhq_prepare, dhq_calibrate, dhq_calibrate_layer, dhq_get_act_absmax, dhq_set_act_absmax, dhq_forward, dhq_forward_host, dhq_forward_debug, dhq_forward_static_scratch,
    DHQ_STATIC_MAX_TOKENS, dhq_get_layer,
    dhq_layer_dims, dhq_last_status, dhq_launch_count, dhq_destroy, dhq_status_string,
    dhq_measure_pipe, library_path, load_library, dhq_forward_fused_debug, dhq_set_wait_limit,
    dhq_debug_stall_next_forward, dhq_measure_sine_error, dhq_export, dhq_import, dhq_last_launch_clock, DHQ_ROT_BOTH, DHQ_ROT_NONE, DHQ_BITS_FLOAT, DHQ_ACT_SINE, DHQ_ACT_GABOR,
)
from .sharded import calibrate_sharded, shard_range  # noqa: F401,E402
